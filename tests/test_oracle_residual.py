"""Pins of the oracle's residual-block coupling network (Eq. 3 of Sec. 4.1 with the scatter add of
Sec. 4.5): a block worked out independently with exact rational arithmetic, identity blocks that
must reduce the network to a plain two-conv chain, the equivalence of a gated full-width second conv
with its compact form plus index list (Eq. 8 + SAdd), and the flow's invariants."""
import copy
from fractions import Fraction
import math

import numpy as np

import iodf_synth as S
import oracle as O


def _rq(a, m0, s):
    return math.floor(Fraction(int(a) * int(m0), 1 << (31 + int(s))) + Fraction(1, 2))


def _layer(w, bias, m0, s, relu, clamp):
    w = np.asarray(w, dtype=np.int8)
    return {"k": w.shape[1], "c_in": w.shape[3], "c_out": w.shape[0], "w": w, "bias": np.asarray(bias, np.int32),
            "m0": np.asarray(m0, np.int32), "s": np.asarray(s, np.int32), "relu": relu, "clamp": clamp, "gate": None}


def test_one_block_by_hand_on_a_single_pixel():
    """3x2x2 image -> 12 channels at 1x1: every 3x3 conv is its centre tap, a matrix product.
    x_a (6 ch) -> conv_in (D = 4) -> one block (K = 3 hidden, K' = 2 kept outputs at channels 1 and 3)
    -> conv_out (6 ch). The expected translation is computed here from Eq. 3 with Fractions."""
    rng = np.random.default_rng(7)
    ca = cb = 6
    D, K, K2 = 4, 3, 2
    idx = [1, 3]

    def rand_layer(cout, cin, relu, clamp, s):
        w = rng.integers(-127, 128, (cout, 3, 3, cin)).astype(np.int8)
        return _layer(w, rng.integers(-500, 500, cout), rng.integers(1 << 30, 1 << 31, cout), np.full(cout, s), relu, clamp)
    conv_in = rand_layer(D, ca, True, (0, 255), 6)
    conv_a = rand_layer(K, D, True, (0, 255), 7)
    conv_b = rand_layer(K2, K, False, None, 7)
    conv_out = rand_layer(cb, D, False, None, 6)
    block = {"short_m0": int(rng.integers(1 << 30, 1 << 31)), "short_s": 0, "clamp": (0, 255), "idx": np.array(idx, np.int32)}
    in_m0, in_s = int(rng.integers(1 << 30, 1 << 31)), 1
    model = {"in_c": 3, "in_h": 2, "in_w": 2, "levels": [{
        "c": 12, "h": 1, "w": 1, "split": False, "prior": None,
        "couplings": [{"perm": np.arange(12, dtype=np.int32), "in_m0": in_m0, "in_s": in_s,
                       "layers": [conv_in, conv_a, conv_b, conv_out], "blocks": [block]}]}]}
    x = rng.integers(0, 256, (1, 3, 2, 2)).astype(np.uint8)
    v = np.array([x[0, c, dy, dx] for c in range(3) for dy in range(2) for dx in range(2)], dtype=np.int64)  # squeeze
    xa, xb = v[:6], v[6:]

    def dense(layer, a):
        out = []
        for o in range(layer["c_out"]):
            acc = int(layer["bias"][o]) + sum(int(layer["w"][o, 1, 1, c]) * int(a[c]) for c in range(layer["c_in"]))
            y = _rq(acc, layer["m0"][o], layer["s"][o])
            if layer["relu"]:
                y = max(y, 0)
            if layer["clamp"] is not None:
                y = min(max(y, layer["clamp"][0]), layer["clamp"][1])
            out.append(y)
        return out
    a0 = [min(max(_rq(t, in_m0, in_s), -128), 127) for t in xa]
    h = dense(conv_in, a0)
    mid = dense(conv_a, h)
    br = dense(conv_b, mid)
    s = [_rq(hc, block["short_m0"], block["short_s"]) for hc in h]          # Q(x) on all D channels
    for j, c in enumerate(idx):
        s[c] += br[j]                                                        # scatter add
    h = [min(max(max(t, 0), 0), 255) for t in s]                            # ReLU, clip
    t = dense(conv_out, h)
    want = np.concatenate([xa, (xb + np.array(t)) & 0xFFFFFFFF]).astype(np.uint32).astype(np.int64)
    z, _ = O.forward(O.Packed(model), x)
    got = z[0].astype(np.int64) & 0xFFFFFFFF
    np.testing.assert_array_equal(got, want)


def test_identity_blocks_reduce_to_the_two_conv_chain():
    """Second conv all zero and a shortcut multiplier of (2^31 - 1) / 2^31 at shift 0: rq(x) = x for
    0 <= x <= 255, so every block is the identity and the network is conv_in -> conv_out."""
    model = S.make_residual_model(11, 3, 8, 8, [True, False], 2, 12, 3, prune=(0.4, 0.8))
    chain = copy.deepcopy(model)
    for lv_r, lv_c in zip(model["levels"], chain["levels"]):
        for cp_r, cp_c in zip(lv_r["couplings"], lv_c["couplings"]):
            for b, rb in enumerate(cp_r["blocks"]):
                second = cp_r["layers"][2 + 2 * b]
                second["w"][:] = 0
                second["bias"][:] = 0
                rb["short_m0"], rb["short_s"] = (1 << 31) - 1, 0
            cp_c["layers"] = [cp_c["layers"][0], cp_c["layers"][-1]]
            cp_c["blocks"] = []
    x = S.smooth_field_images(12, 3, 8, 8, 1.5)
    z_res, p_res = O.forward(O.Packed(model), x)
    z_chain, p_chain = O.forward(O.Packed(chain), x)
    np.testing.assert_array_equal(z_res, z_chain)
    np.testing.assert_array_equal(p_res, p_chain)


def test_gated_full_width_second_conv_equals_compact_with_index_list():
    """Eq. 8: a filter whose gate is 0 outputs zero; Sec. 4.5: the scatter add puts the kept outputs
    back at their channels. A block whose second conv has all D filters with gates, placed by the
    identity index list, must equal the compact block (kept filters only + their index list)."""
    model = S.make_residual_model(21, 3, 8, 8, [True], 2, 10, 2, prune=(0.4, 0.7))
    dense = copy.deepcopy(model)
    rng = np.random.default_rng(22)
    for cp in dense["levels"][0]["couplings"]:
        D = cp["layers"][0]["c_out"]
        for b, rb in enumerate(cp["blocks"]):
            ly = cp["layers"][2 + 2 * b]
            k2, k1 = ly["c_out"], ly["c_in"]
            idx = rb["idx"]
            w = rng.integers(-127, 128, (D, 3, 3, k1)).astype(np.int8)       # pruned filters: anything
            bias = rng.integers(-1000, 1000, D).astype(np.int32)
            m0 = rng.integers(1 << 30, 1 << 31, D).astype(np.int32)
            s = rng.integers(0, 12, D).astype(np.int32)
            gate = np.zeros(D, np.int32)
            w[idx], bias[idx], m0[idx], s[idx], gate[idx] = ly["w"], ly["bias"], ly["m0"], ly["s"], 1
            ly.update({"c_out": D, "w": w, "bias": bias, "m0": m0, "s": s, "gate": gate})
            rb["idx"] = np.arange(D, dtype=np.int32)
    x = S.smooth_field_images(23, 4, 8, 8, 1.5)
    z_c, p_c = O.forward(O.Packed(model), x)
    z_d, p_d = O.forward(O.Packed(dense), x)
    np.testing.assert_array_equal(z_c, z_d)
    np.testing.assert_array_equal(p_c, p_d)
    # and the gates matter: opening them changes z
    for cp in dense["levels"][0]["couplings"]:
        for b in range(len(cp["blocks"])):
            cp["layers"][2 + 2 * b]["gate"][:] = 1
    assert not np.array_equal(O.forward(O.Packed(dense), x)[0], z_c)


def test_residual_flow_invariants():
    """Bijection in both directions, prior parameters identical in both, blocks really contribute."""
    model = S.make_residual_model(31, 3, 16, 16, [True, True, True], 2, 24, 3, prune=(0.4, 0.7))
    pk = O.Packed(model)
    x = np.concatenate([S.smooth_field_images(32, 3, 16, 16, 2.0), np.zeros((1, 3, 16, 16), np.uint8),
                        np.full((1, 3, 16, 16), 255, np.uint8)])
    z, p = O.forward(pk, x)
    xu, xi, p2, oor = O.inverse(pk, z)
    np.testing.assert_array_equal(xu, x)
    np.testing.assert_array_equal(p, p2)
    assert oor == 0
    rng = np.random.default_rng(33)
    zr = rng.integers(-2**31, 2**31, z.shape).astype(np.int32)
    _, xi, _, _ = O.inverse(pk, zr)
    # forward takes uint8 images only; the bijection on arbitrary latents is checked where x stays in range
    inr = np.all((xi >= 0) & (xi <= 255), axis=(1, 2, 3))
    if inr.any():
        np.testing.assert_array_equal(O.forward(pk, xi[inr].astype(np.uint8))[0], zr[inr])
    # dropping the blocks changes the result (they are not dead code)
    chain = copy.deepcopy(model)
    for lv in chain["levels"]:
        for cp in lv["couplings"]:
            cp["layers"] = [cp["layers"][0], cp["layers"][-1]]
            cp["blocks"] = []
    assert not np.array_equal(O.forward(O.Packed(chain), x)[0], z)
    # a malformed block (index list with a repeated channel) is rejected
    bad = copy.deepcopy(model)
    bad["levels"][0]["couplings"][0]["blocks"][0]["idx"][:2] = 0
    try:
        O.Packed(bad)
        assert False, "repeated index accepted"
    except ValueError:
        pass
