"""Seeded IODF model descriptions: level/coupling structure, pruned hidden widths, int8 weights,
int32 biases and per-output-channel fixed-point requantisation pairs (M0, s).

A model is a plain dict:

  {"in_c", "in_h", "in_w", "levels": [level, ...]}
  level    = {"c", "h", "w", "couplings": [coupling, ...], "split": bool, "prior": head | None}
  coupling = {"perm": int32[c], "in_m0": int, "in_s": int, "layers": [layer, ...]}
  layer    = {"k": 1 | 3, "c_in", "c_out", "w": int8[c_out, k, k, c_in], "bias": int32[c_out],
              "m0": int32[c_out], "s": int32[c_out], "relu": bool,
              "clamp": (lo, hi) | None, "gate": uint8[c_out] | None}
  head     = {"in_m0", "in_s", "layer": layer (c/2 -> c: first half mu, second half ls),
              "ls_lo", "ls_hi"}

Only shapes and random draws live here; what the numbers mean is defined by the code that
consumes them.
"""
import math

import numpy as np

from .rng import Stream
from .images import smooth_field_images

SIGMA_W = 32.0


def level_shapes(in_c, in_h, in_w, splits):
    """[(c, h, w)] per level: a 2x2 space-to-depth before each level, channel halving at a split."""
    shapes = []
    c, h, w = in_c, in_h, in_w
    for sp in splits:
        c, h, w = c * 4, h // 2, w // 2
        shapes.append((c, h, w))
        if sp:
            c //= 2
    return shapes


def _shift_for(fan_in, rms_in):
    v = math.log2(0.75 * SIGMA_W * rms_in * math.sqrt(fan_in) / 32.0)
    return int(min(31, max(0, math.floor(v + 0.5))))


def _layer(st, k, c_in, c_out, rms_in, relu, clamp, with_bias):
    fan_in = k * k * c_in
    w = np.clip(np.floor(st.normal(c_out * fan_in) * SIGMA_W + 0.5), -127, 127)
    w = w.astype(np.int8).reshape(c_out, k, k, c_in)
    sigma_acc = SIGMA_W * rms_in * math.sqrt(fan_in)
    nb = st.normal(c_out)
    bias = (np.floor(nb * (sigma_acc / 4.0) + 0.5) if with_bias else np.zeros(c_out)).astype(np.int32)
    m0 = st.integers(1 << 30, 1 << 31, c_out).astype(np.int32)
    s = np.full(c_out, _shift_for(fan_in, rms_in), dtype=np.int32)
    return {"k": k, "c_in": c_in, "c_out": c_out, "w": w, "bias": bias, "m0": m0, "s": s,
            "relu": relu, "clamp": clamp, "gate": None}


def make_model(seed, in_c, in_h, in_w, splits, n_couplings, hidden, prune=None, prior=True,
               perm="random", act_hi=127, with_bias=True):
    """splits: one bool per level. prune: None or (lo, hi) keep-fraction range; kept widths are
    made odd. perm: "random" (seeded Fisher-Yates per coupling) or "reverse" (identity before the
    first coupling of a level, channel reversal before the others)."""
    shapes = level_shapes(in_c, in_h, in_w, splits)
    levels = []
    for li, ((c, h, w), sp) in enumerate(zip(shapes, splits)):
        if c % 2 or h < 1 or w < 1:
            raise ValueError("bad level shape")
        ca, cb = c // 2, c - c // 2
        couplings = []
        for ki in range(n_couplings):
            st = Stream(seed, "L%d/K%d" % (li, ki))
            if perm == "random":
                p = st.permutation(c)
            else:
                p = np.arange(c) if ki == 0 else np.arange(c)[::-1].copy()
            if prune is None:
                k1 = k2 = hidden
            else:
                f = prune[0] + (prune[1] - prune[0]) * st.uniform(2)
                k1, k2 = (int(math.floor(hidden * x + 0.5)) | 1 for x in f)
            layers = [
                _layer(st, 3, ca, k1, 48.0, True, (0, act_hi), with_bias),
                _layer(st, 1, k1, k2, 23.0, True, (0, act_hi), with_bias),
                _layer(st, 3, k2, cb, 23.0, False, None, with_bias),
            ]
            couplings.append({"perm": p.astype(np.int32),
                              "in_m0": int(st.integers(1 << 30, 1 << 31, 1)[0]), "in_s": 1,
                              "layers": layers})
        head = None
        if sp and prior:
            st = Stream(seed, "L%d/prior" % li)
            head = {"in_m0": int(st.integers(1 << 30, 1 << 31, 1)[0]), "in_s": 1,
                    "layer": _layer(st, 3, ca, 2 * cb, 48.0, False, None, with_bias),
                    "ls_lo": 0, "ls_hi": 63}
        levels.append({"c": c, "h": h, "w": w, "couplings": couplings, "split": bool(sp),
                       "prior": head})
    return {"in_c": in_c, "in_h": in_h, "in_w": in_w, "levels": levels}


def make_residual_model(seed, in_c, in_h, in_w, splits, n_couplings, hidden, n_blocks, prune=None, prior=True):
    """The flow with the paper's coupling network: conv3x3 (C/2 -> hidden), n_blocks residual blocks
    [conv3x3 (hidden -> K), ReLU, conv3x3 (K -> K'), scatter add onto the hidden-wide shortcut, ReLU],
    conv3x3 (hidden -> C/2). K, K' are the kept (odd) widths when `prune` = (lo, hi) keep fractions.
    A coupling carries "blocks": per block the shortcut requantisation pair, the clip after the ReLU
    and the index list that places the second conv's K' outputs among the hidden channels.
    Hidden activations use the unsigned 8-bit range 0..255."""
    shapes = level_shapes(in_c, in_h, in_w, splits)
    levels = []
    for li, ((c, h, w), sp) in enumerate(zip(shapes, splits)):
        ca, cb = c // 2, c - c // 2
        couplings = []
        for ki in range(n_couplings):
            st = Stream(seed, "R%d/K%d" % (li, ki))
            p = st.permutation(c)
            layers = [_layer(st, 3, ca, hidden, 48.0, True, (0, 255), True)]
            blocks = []
            for b in range(n_blocks):
                if prune is None:
                    k1 = k2 = hidden
                else:
                    f = prune[0] + (prune[1] - prune[0]) * st.uniform(2)
                    k1, k2 = (min(hidden, int(math.floor(hidden * x + 0.5)) | 1) for x in f)
                layers.append(_layer(st, 3, hidden, k1, 23.0, True, (0, 255), True))
                layers.append(_layer(st, 3, k1, k2, 23.0, False, None, True))
                idx = np.sort(st.permutation(hidden)[:k2]).astype(np.int32)
                blocks.append({"short_m0": int(st.integers(1 << 30, 1 << 31, 1)[0]), "short_s": 0,
                               "clamp": (0, 255), "idx": idx})
            layers.append(_layer(st, 3, hidden, cb, 30.0, False, None, True))
            couplings.append({"perm": p.astype(np.int32), "in_m0": int(st.integers(1 << 30, 1 << 31, 1)[0]),
                              "in_s": 1, "layers": layers, "blocks": blocks})
        head = None
        if sp and prior:
            st = Stream(seed, "R%d/prior" % li)
            head = {"in_m0": int(st.integers(1 << 30, 1 << 31, 1)[0]), "in_s": 1,
                    "layer": _layer(st, 3, ca, 2 * cb, 48.0, False, None, True), "ls_lo": 0, "ls_hi": 63}
        levels.append({"c": c, "h": h, "w": w, "couplings": couplings, "split": bool(sp), "prior": head})
    return {"in_c": in_c, "in_h": in_h, "in_w": in_w, "levels": levels}


def latent_sizes(model):
    """(d, d_fact, blocks): blocks = [(level, channels, h, w, has_prior)] in z order."""
    blocks = []
    for li, lv in enumerate(model["levels"]):
        if lv["split"]:
            blocks.append((li, lv["c"] - lv["c"] // 2, lv["h"], lv["w"], lv["prior"] is not None))
    last = model["levels"][-1]
    blocks.append((len(model["levels"]) - 1, last["c"] // 2 if last["split"] else last["c"],
                   last["h"], last["w"], False))
    d = sum(c * h * w for _, c, h, w, _ in blocks)
    d_fact = sum(c * h * w for _, c, h, w, p in blocks if p)
    return d, d_fact, blocks


def model_macs(model):
    """Multiply-accumulates per image over the kept channels (unpadded)."""
    total = 0
    for lv in model["levels"]:
        px = lv["h"] * lv["w"]
        for cp in lv["couplings"]:
            for ly in cp["layers"]:
                total += px * ly["k"] ** 2 * ly["c_in"] * ly["c_out"]
        if lv["prior"] is not None:
            ly = lv["prior"]["layer"]
            total += px * ly["k"] ** 2 * ly["c_in"] * ly["c_out"]
    return total


def _copy_layer(ly):
    return {k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in ly.items()}


def _copy_model(model, fn):
    out = {k: model[k] for k in ("in_c", "in_h", "in_w")}
    out["levels"] = []
    for li, lv in enumerate(model["levels"]):
        nl = dict(lv)
        nl["couplings"] = []
        for ki, cp in enumerate(lv["couplings"]):
            nc = dict(cp)
            nc["perm"] = cp["perm"].copy()
            nc["layers"] = fn(li, ki, [_copy_layer(l) for l in cp["layers"]])
            nl["couplings"].append(nc)
        if lv["prior"] is not None:
            nl["prior"] = dict(lv["prior"])
            nl["prior"]["layer"] = _copy_layer(lv["prior"]["layer"])
        out["levels"].append(nl)
    return out


def _widen(layers, idx, new_w, positions, fill_st):
    """Grow the output of layers[idx] (and the matching input of layers[idx+1]) to new_w channels,
    placing the existing channels at `positions`. New filters get `fill_st` draws (or zeros)."""
    a, b = layers[idx], layers[idx + 1]
    old = a["c_out"]
    k = a["k"]

    def draw(shape):
        if fill_st is None:
            return np.zeros(shape, dtype=np.int8)
        n = int(np.prod(shape))
        return np.clip(np.floor(fill_st.normal(n) * SIGMA_W + 0.5), -127, 127).astype(np.int8).reshape(shape)

    w = draw((new_w, k, k, a["c_in"]))
    w[positions] = a["w"]
    bias = (np.zeros(new_w) if fill_st is None else np.floor(fill_st.normal(new_w) * 500 + 0.5)).astype(np.int32)
    bias[positions] = a["bias"]
    m0 = np.full(new_w, 1 << 30, dtype=np.int32)
    m0[positions] = a["m0"]
    s = np.zeros(new_w, dtype=np.int32) if fill_st is None else np.full(new_w, int(a["s"][0]), np.int32)
    s[positions] = a["s"]
    gate = np.zeros(new_w, dtype=np.uint8)
    gate[positions] = 1
    a.update(c_out=new_w, w=w, bias=bias, m0=m0, s=s, gate=None if fill_st is None else gate)
    wb = draw((b["c_out"], b["k"], b["k"], new_w))
    wb[..., positions] = b["w"]
    b.update(c_in=new_w, w=wb)
    assert old == len(positions)


def masked_dense_model(model, seed, hidden):
    """The same function as `model`, written as a dense width-`hidden` network whose extra
    filters carry random weights and biases but a zero gate."""
    def fn(li, ki, layers):
        st = Stream(seed, "dense/L%d/K%d" % (li, ki))
        for idx in range(len(layers) - 1):
            old = layers[idx]["c_out"]
            pos = np.sort(st.permutation(hidden)[:old])
            _widen(layers, idx, hidden, pos, st)
        return layers
    return _copy_model(model, fn)


def zero_padded_model(model, multiple):
    """The same function as `model` with every hidden width rounded up to `multiple` by appending
    channels with zero weights, zero bias and (M0, s) = (2^30, 0)."""
    def fn(li, ki, layers):
        for idx in range(len(layers) - 1):
            old = layers[idx]["c_out"]
            new_w = -(-old // multiple) * multiple
            _widen(layers, idx, new_w, np.arange(old), None)
        return layers
    return _copy_model(model, fn)


# The five benchmark configurations: shapes, batch, blur, pruning law, seeds.
CONFIGS = {
    0: dict(seed=0x10DF0000, batch=16, hw=32, sigma=2.0, splits=[False], n_couplings=4, hidden=64,
            prune=None, prior=False, perm="reverse"),
    1: dict(seed=0x10DF0001, batch=256, hw=32, sigma=2.0, splits=[True] * 3, n_couplings=8,
            hidden=256, prune=(0.40, 0.70), prior=True, perm="random"),
    2: dict(seed=0x10DF0002, batch=128, hw=64, sigma=4.0, splits=[True] * 4, n_couplings=8,
            hidden=256, prune=(0.40, 0.70), prior=True, perm="random"),
    3: dict(seed=0x10DF0001, batch=256, hw=32, sigma=2.0, splits=[True] * 3, n_couplings=8,
            hidden=256, prune=(0.40, 0.70), prior=True, perm="random"),
    4: dict(seed=0x10DF0002, batch=64, hw=64, sigma=4.0, splits=[True] * 4, n_couplings=8,
            hidden=256, prune=(0.40, 0.70), prior=True, perm="random"),
    "4s": dict(seed=0x10DF0004, batch=64, hw=64, sigma=4.0, splits=[True] * 4, n_couplings=8,
               hidden=512, prune=None, prior=True, perm="random"),
    # the paper's own coupling network (App. B.1) on the ImageNet32 geometry: 3 levels x 8 couplings,
    # each conv3x3 -> 8 gated residual blocks -> conv3x3 on 128 hidden channels, about half pruned
    "R32": dict(seed=0x10DF0032, batch=64, hw=32, sigma=2.0, splits=[True] * 3, n_couplings=8,
                hidden=128, prune=(0.40, 0.70), prior=True, perm="random", n_blocks=8),
    # the same network on the ImageNet64 geometry (Sec. 5, App. B.1): 4 levels, the first of 32 x 32 pixels
    "R64": dict(seed=0x10DF0064, batch=32, hw=64, sigma=4.0, splits=[True] * 4, n_couplings=8,
                hidden=128, prune=(0.40, 0.70), prior=True, perm="random", n_blocks=8),
}


def config_model(idx):
    c = CONFIGS[idx]
    if c.get("n_blocks"):
        return make_residual_model(c["seed"], 3, c["hw"], c["hw"], c["splits"], c["n_couplings"], c["hidden"],
                                   c["n_blocks"], prune=c["prune"], prior=c["prior"])
    return make_model(c["seed"], 3, c["hw"], c["hw"], c["splits"], c["n_couplings"], c["hidden"],
                      prune=c["prune"], prior=c["prior"], perm=c["perm"])


def config_images(idx, batch=None, seed_offset=0):
    c = CONFIGS[idx]
    return smooth_field_images(c["seed"] + 0x1000 + seed_offset, batch or c["batch"], c["hw"], c["hw"],
                               c["sigma"])
