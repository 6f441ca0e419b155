"""Pins for the CPU oracle: each part is checked against something other than itself -- exact
rational arithmetic, a library correlation routine, closed-form index maps, the bijection
invariant of Eq. 2, the pruning equivalence of Eq. 8, and a hand-worked example."""
import os
from fractions import Fraction
import math

import numpy as np
import pytest
from scipy.signal import correlate2d

import iodf_synth as S
import oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---- requantisation: Eq. "quant_conv" with the multiplier M0 * 2^-(31+s), ties toward +inf -------
def _rq_exact(a, m0, s):
    return math.floor(Fraction(a * m0, 1 << (31 + s)) + Fraction(1, 2))


def test_rq_hand_cases():
    half = 1 << 30  # multiplier exactly 1/2
    for a, want in [(1, 1), (-1, 0), (3, 2), (-3, -1), (0, 0), (2, 1), (-2, -1), (255, 128)]:
        assert O.rq(a, half, 0) == want
    assert O.rq(4, half, 1) == 1       # 4 * 1/4
    assert O.rq(2, half, 1) == 1       # 0.5 rounds up
    assert O.rq(-2, half, 1) == 0      # -0.5 rounds up to 0
    assert O.rq(-6, half, 1) == -1     # -1.5 rounds up to -1


def test_rq_matches_rational_rounding():
    st = S.Stream(11, "rq")
    n = 200000
    a = st.integers(-(1 << 31), 1 << 31, n)
    m0 = st.integers(1 << 30, 1 << 31, n)
    s = st.integers(0, 32, n)
    # exact ties and range ends
    extra = [((1 << 31) - 1, (1 << 31) - 1, 0), (-(1 << 31), (1 << 31) - 1, 0), ((1 << 31) - 1, 1 << 30, 31),
             (-(1 << 31), 1 << 30, 31), (1, 1 << 30, 0), (-1, 1 << 30, 0)]
    for sh in range(32):
        for kk in (-5, -1, 1, 3, 7):
            extra.append((kk * (1 << sh), 1 << 30, sh))  # a*M0 = odd multiple of 2^(30+s): exact .5
    for ai, mi, si in list(zip(a.tolist(), m0.tolist(), s.tolist())) + extra:
        got = O.rq(ai, mi, si)
        assert got == _rq_exact(ai, mi, si), (ai, mi, si)


def test_rq_within_half_of_real_value():
    st = S.Stream(12, "rq-real")
    for ai, mi, si in zip(st.integers(-(1 << 24), 1 << 24, 2000).tolist(),
                          st.integers(1 << 30, 1 << 31, 2000).tolist(), st.integers(0, 20, 2000).tolist()):
        real = Fraction(ai * mi, 1 << (31 + si))
        got = O.rq(ai, mi, si)
        assert Fraction(-1, 2) < got - real <= Fraction(1, 2)


# ---- convolution: Eq. 5, stride 1, zero padding, shape preserved ------------------------------
def _ref_conv(w, bias, x):
    """Sum over input channels of library 2-D cross-correlations ('same', zero fill) plus bias."""
    c_out, k, _, c_in = w.shape
    out = np.zeros((c_out,) + x.shape[1:], dtype=np.int64)
    for co in range(c_out):
        for ci in range(c_in):
            out[co] += correlate2d(x[ci].astype(np.int64), w[co, :, :, ci].astype(np.int64), mode="same",
                                   boundary="fill", fillvalue=0)
        out[co] += int(bias[co])
    return out


@pytest.mark.parametrize("h,w", [(1, 1), (1, 2), (2, 1), (2, 2), (3, 5), (8, 8)])
@pytest.mark.parametrize("k", [1, 3])
def test_conv_matches_library_correlation(h, w, k):
    st = S.Stream(21, "conv%d%d%d" % (h, w, k))
    c_in, c_out = 3, 4
    wt = st.integers(-127, 128, c_out * k * k * c_in).astype(np.int8).reshape(c_out, k, k, c_in)
    bias = st.integers(-1000, 1000, c_out).astype(np.int32)
    x = st.integers(-128, 128, c_in * h * w).astype(np.int32).reshape(c_in, h, w)
    np.testing.assert_array_equal(O.conv_acc(wt, bias, x), _ref_conv(wt, bias, x))


def test_conv_single_pixel_is_centre_tap_dot_product():
    st = S.Stream(22, "centre")
    wt = st.integers(-127, 128, 5 * 9 * 7).astype(np.int8).reshape(5, 3, 3, 7)
    x = st.integers(-128, 128, 7).astype(np.int32).reshape(7, 1, 1)
    bias = np.arange(5, dtype=np.int32)
    want = wt[:, 1, 1, :].astype(np.int64) @ x.reshape(7).astype(np.int64) + bias
    np.testing.assert_array_equal(O.conv_acc(wt, bias, x).reshape(5), want)


def test_conv_1x1_is_matrix_product_and_linear():
    st = S.Stream(23, "1x1")
    wt = st.integers(-127, 128, 6 * 5).astype(np.int8).reshape(6, 1, 1, 5)
    x = st.integers(-128, 128, 5 * 12).astype(np.int32).reshape(5, 3, 4)
    y = st.integers(-128, 128, 5 * 12).astype(np.int32).reshape(5, 3, 4)
    zero = np.zeros(6, np.int32)
    want = np.einsum("oc,chw->ohw", wt.reshape(6, 5).astype(np.int64), x.astype(np.int64))
    np.testing.assert_array_equal(O.conv_acc(wt, zero, x), want)
    w3 = st.integers(-127, 128, 6 * 9 * 5).astype(np.int8).reshape(6, 3, 3, 5)
    np.testing.assert_array_equal(O.conv_acc(w3, zero, x + y), O.conv_acc(w3, zero, x) + O.conv_acc(w3, zero, y))


def test_conv_reports_int32_overflow():
    wt = np.full((1, 3, 3, 4096), 127, np.int8)
    x = np.full((4096, 1, 1), 127, np.int32)
    O.conv_acc(wt, np.zeros(1, np.int32), x)          # 4096*127*127 fits
    with pytest.raises(RuntimeError):
        O.conv_acc(wt, np.full(1, 2**31 - 1, np.int32), x)


# ---- index maps: squeeze, permutation, split and latent layout, closed form ---------------------
def test_squeeze_closed_form_and_inverse():
    x = np.arange(3 * 4 * 6, dtype=np.int32).reshape(3, 4, 6)
    y = O.squeeze(x)
    assert y.shape == (12, 2, 3)
    for c in range(3):
        for dy in range(2):
            for dx in range(2):
                np.testing.assert_array_equal(y[c * 4 + dy * 2 + dx], x[c, dy::2, dx::2])
    np.testing.assert_array_equal(O.unsqueeze(y), x)


def _zero_model(model):
    for lv in model["levels"]:
        for cp in lv["couplings"]:
            for ly in cp["layers"]:
                ly["w"][:] = 0
                ly["bias"][:] = 0
    return model


def _rearrange_closed_form(model, x):
    """What z must be when every translation is zero: squeeze, permute, split, concatenate."""
    v = x.astype(np.int32)
    blocks = []
    for lv in model["levels"]:
        c, h, w = v.shape
        v = v.reshape(c, h // 2, 2, w // 2, 2).transpose(0, 2, 4, 1, 3).reshape(c * 4, h // 2, w // 2)
        for cp in lv["couplings"]:
            v = v[cp["perm"]]
        if lv["split"]:
            half = v.shape[0] // 2
            blocks.append(v[half:].reshape(-1))
            v = v[:half]
    blocks.append(v.reshape(-1))
    return np.concatenate(blocks)


@pytest.mark.parametrize("splits", [[True, True], [True, False], [False]])
def test_zero_translation_gives_pure_rearrangement(splits):
    model = _zero_model(S.make_model(5, 3, 8, 8, splits, 3, 7, prune=None, prior=True))
    x = S.smooth_field_images(6, 4, 8, 8, 1.0)
    z, _ = O.forward(O.Packed(model), x)
    for b in range(4):
        np.testing.assert_array_equal(z[b], _rearrange_closed_form(model, x[b]))
    d, d_fact, blocks = S.latent_sizes(model)
    assert z.shape[1] == d == 3 * 8 * 8


def test_constant_translation_pins_sign_and_updated_half():
    """Zero weights but a non-zero last-layer bias: t = rq(bias) everywhere, so z_b - x_b is that
    constant, z_a = x_a, and the inverse subtracts it again."""
    model = _zero_model(S.make_model(7, 1, 2, 2, [False], 1, 3, prune=None, prior=False, perm="reverse"))
    last = model["levels"][0]["couplings"][0]["layers"][-1]
    last["bias"][:] = [1000, -777]
    want_t = [_rq_exact(int(b), int(m), int(s)) for b, m, s in zip(last["bias"], last["m0"], last["s"])]
    x = np.array([[[[10, 20], [30, 40]]]], dtype=np.uint8)
    z, _ = O.forward(O.Packed(model), x)
    np.testing.assert_array_equal(z[0], [10, 20, 30 + want_t[0], 40 + want_t[1]])
    xu, xi, _, oor = O.inverse(O.Packed(model), z)
    np.testing.assert_array_equal(xi, x.astype(np.int32))


def _golden_rows(name):
    rows = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, *v = line.split()
                rows[k] = [int(t) for t in v]
    return rows


def _two_layer_model(w1, b1, w2, b2):
    half = dict(m0=np.full(2, 1 << 30, np.int32), s=np.zeros(2, np.int32), gate=None)
    l1 = dict(k=1, c_in=2, c_out=2, w=np.array(w1, np.int8).reshape(2, 1, 1, 2),
              bias=np.array(b1, np.int32), relu=True, clamp=(0, 127), **half)
    l2 = dict(k=1, c_in=2, c_out=2, w=np.array(w2, np.int8).reshape(2, 1, 1, 2),
              bias=np.array(b2, np.int32), relu=False, clamp=None, **half)
    cp = dict(perm=np.arange(4, dtype=np.int32), in_m0=1 << 30, in_s=0, layers=[l1, l2])
    return dict(in_c=1, in_h=2, in_w=2, levels=[dict(c=4, h=1, w=1, couplings=[cp], split=False, prior=None)])


@pytest.mark.parametrize("name,w1,b1,w2,b2", [
    ("hand_coupling.txt", [[1, -1], [2, 0]], [3, -4], [[5, 7], [-3, 1]], [1, 1]),
    ("hand_saturation.txt", [[127, 0], [-1, 0]], [0, 0], [[1, 0], [0, 1]], [0, 0]),
])
def test_hand_worked_coupling(name, w1, b1, w2, b2):
    rows = _golden_rows(name)
    model = _two_layer_model(w1, b1, w2, b2)
    x = np.array(rows["x"], np.uint8).reshape(1, 1, 2, 2)   # squeeze order: (0,0),(0,1),(1,0),(1,1)
    z, _ = O.forward(O.Packed(model), x)
    assert z[0].tolist() == rows["z"]
    xu, _, _, _ = O.inverse(O.Packed(model), z)
    np.testing.assert_array_equal(xu, x)


# ---- the bijection (Sec. 3: p_X(x) = p_Z(f(x)) needs f invertible on Z^d) -----------------------
@pytest.mark.parametrize("cfg", [
    dict(splits=[True, True, True], hidden=24, prune=(0.4, 0.7), hw=16),
    dict(splits=[True, False], hidden=16, prune=None, hw=8),
    dict(splits=[False], hidden=9, prune=None, hw=4),
])
def test_round_trip_both_ways(cfg):
    model = S.make_model(31, 3, cfg["hw"], cfg["hw"], cfg["splits"], 4, cfg["hidden"], prune=cfg["prune"])
    pk = O.Packed(model)
    hw = cfg["hw"]
    x = np.concatenate([S.smooth_field_images(32, 5, hw, hw, 1.5),
                        np.zeros((1, 3, hw, hw), np.uint8), np.full((1, 3, hw, hw), 255, np.uint8),
                        S.Stream(33, "u8").integers(0, 256, 3 * hw * hw).astype(np.uint8).reshape(1, 3, hw, hw)])
    z, prior = O.forward(pk, x)
    xu, xi, prior2, oor = O.inverse(pk, z)
    np.testing.assert_array_equal(xu, x)
    np.testing.assert_array_equal(xi, x.astype(np.int32))
    assert oor == 0
    if prior is not None:
        np.testing.assert_array_equal(prior, prior2)
    # any integer vector is a valid latent: inverse then forward returns it (arithmetic wraps mod 2^32)
    zr = S.Stream(34, "z").integers(-(1 << 31), 1 << 31, 3 * pk.d).astype(np.int32).reshape(3, pk.d)
    _, xi2, _, _ = O.inverse(pk, zr, want_prior=False)
    # forward takes u8 only, so check the small-range case through u8 and the wide case by trace-free identity
    zs = S.Stream(35, "zs").integers(-40, 40, 2 * pk.d).astype(np.int32).reshape(2, pk.d)
    xu3, xi3, _, _ = O.inverse(pk, zs, want_prior=False)
    inr = np.all((xi3 >= 0) & (xi3 <= 255), axis=(1, 2, 3))
    if inr.any():
        z3, _ = O.forward(pk, xu3[inr], want_prior=False)
        np.testing.assert_array_equal(z3, zs[inr])
    assert xi2.shape == (3, 3, hw, hw)


def test_batch_position_independence():
    model = S.make_model(41, 3, 8, 8, [True, True], 2, 12, prune=(0.4, 0.7))
    pk = O.Packed(model)
    x = S.smooth_field_images(42, 6, 8, 8, 1.0)
    z, p = O.forward(pk, x)
    z1, p1 = O.forward(pk, x[3:4], threads=1)
    np.testing.assert_array_equal(z[3:4], z1)
    np.testing.assert_array_equal(p[3:4], p1)
    zr, pr = O.forward(pk, x[::-1])
    np.testing.assert_array_equal(zr[::-1], z)


def test_trace_ends_in_z():
    model = S.make_model(43, 3, 8, 8, [False], 3, 10, prune=None, prior=False)
    pk = O.Packed(model)
    x = S.smooth_field_images(44, 1, 8, 8, 1.0)
    z, _ = O.forward(pk, x)
    v = O.trace(pk, x[0], 0, 2, (12, 4, 4))
    np.testing.assert_array_equal(v.reshape(-1), z[0])


# ---- pruning (Sec. 4.4, Eq. 8): gated-dense == compact == zero-padded ----------------------------
def test_masked_dense_equals_compact_equals_padded():
    model = S.make_model(51, 3, 8, 8, [True, True], 3, 32, prune=(0.4, 0.7))
    x = S.smooth_field_images(52, 3, 8, 8, 1.0)
    z, p = O.forward(O.Packed(model), x)
    dense = S.masked_dense_model(model, 53, 32)
    assert all(ly["c_out"] == 32 for lv in dense["levels"] for cp in lv["couplings"] for ly in cp["layers"][:-1])
    zd, pd = O.forward(O.Packed(dense), x)
    zp, pp = O.forward(O.Packed(S.zero_padded_model(model, 16)), x)
    np.testing.assert_array_equal(zd, z)
    np.testing.assert_array_equal(zp, z)
    np.testing.assert_array_equal(pd, p)
    # without its gates the dense model is a different function (the gates are what prune)
    for lv in dense["levels"]:
        for cp in lv["couplings"]:
            for ly in cp["layers"]:
                ly["gate"] = None
    zn, _ = O.forward(O.Packed(dense), x)
    assert (zn != z).any()


# ---- ReLU / clip ---------------------------------------------------------------------------------
def test_hidden_activations_saturate_and_prior_scale_is_clipped():
    model = S.make_model(61, 3, 8, 8, [True], 1, 8, prune=None)
    pk = O.Packed(model)
    x = S.smooth_field_images(62, 2, 8, 8, 1.0)
    _, p = O.forward(pk, x)
    hd = model["levels"][0]["prior"]
    assert p[:, 1].min() >= hd["ls_lo"] and p[:, 1].max() <= hd["ls_hi"]
    assert (p[:, 1] == hd["ls_lo"]).any()
    # a huge multiplier on the first layer drives every positive pre-activation to the clip value:
    # the translation then only depends on the sign pattern, and shrinking the clip shrinks |t|
    m2 = S.make_model(61, 3, 8, 8, [True], 1, 8, prune=None, act_hi=1)
    z_hi, _ = O.forward(pk, x)
    z_lo, _ = O.forward(O.Packed(m2), x)
    assert (z_hi != z_lo).any()


def test_bad_descriptors_are_rejected():
    model = S.make_model(71, 3, 4, 4, [False], 1, 4, prune=None, prior=False)
    model["levels"][0]["couplings"][0]["perm"][0] = model["levels"][0]["couplings"][0]["perm"][1]
    with pytest.raises(ValueError):
        O.Packed(model)
    model = S.make_model(71, 3, 4, 4, [False], 1, 4, prune=None, prior=False)
    model["levels"][0]["couplings"][0]["layers"][0]["m0"][0] = 5
    with pytest.raises(ValueError):
        O.Packed(model)


# ---- prior head: (mu, s) of the factored-out half from the kept half (Sec. 3, App. B.1) ---------
def _clip(v, lo, hi):
    return min(max(v, lo), hi)


def test_prior_head_one_pixel_against_rational_arithmetic():
    """A 1x1-pixel level: the head's 3x3 conv is its centre tap, so mu and the log-scale index can be
    written out with exact fractions: input requant with its clip to -128..127 (one kept value is
    large enough to hit 127), dot product, bias, per-channel rq, clip of the log-scale half only."""
    model = _zero_model(S.make_model(81, 1, 2, 2, [True], 1, 3, prune=None, prior=True, perm="reverse"))
    hd = model["levels"][0]["prior"]
    hd["in_m0"], hd["in_s"] = (1 << 31) - 1, 0                 # multiplier just under 1: 255 -> clip at 127
    hd["ls_lo"], hd["ls_hi"] = 2, 9
    ly = hd["layer"]
    st = S.Stream(82, "head")
    ly["w"][:] = st.integers(-127, 128, ly["w"].size).astype(np.int8).reshape(ly["w"].shape)
    ly["bias"][:] = [37, -1200, 2500, -90000]                  # ls biases on both sides of the clip
    ly["m0"][:] = st.integers(1 << 30, 1 << 31, 4).astype(np.int32)
    ly["s"][:] = [3, 5, 4, 2]
    x = np.array([[[[255, 60], [7, 200]]]], dtype=np.uint8)    # squeeze order: 255, 60, 7, 200
    z, p = O.forward(O.Packed(model), x)
    keep = [255, 60]                                           # identity permutation, zero translation
    a = [_clip(_rq_exact(v, hd["in_m0"], hd["in_s"]), -128, 127) for v in keep]
    assert a == [127, 60]
    out = []
    for co in range(4):
        acc = sum(int(ly["w"][co, 1, 1, ci]) * a[ci] for ci in range(2)) + int(ly["bias"][co])
        out.append(_rq_exact(acc, int(ly["m0"][co]), int(ly["s"][co])))
    want_mu = out[:2]
    want_ls = [_clip(v, 2, 9) for v in out[2:]]
    assert out[2] > 9 and out[3] < 2                           # both sides of the clip are exercised
    assert p.shape == (1, 2, 2)
    assert p[0, 0].tolist() == want_mu
    assert p[0, 1].tolist() == want_ls
    assert z[0].tolist() == [7, 200, 255, 60]                  # factored-out half first, kept half last
    _, _, p2, _ = O.inverse(O.Packed(model), z)
    np.testing.assert_array_equal(p2, p)


def test_prior_layout_across_levels_with_constant_heads():
    """Zero weights everywhere and constant head biases: every mu / log-scale index is rq(bias) of
    its channel, so the prior array must be [mu of level 0 | mu of level 1] then [ls of level 0 | ls
    of level 1], each block channel-major over the level's pixels."""
    model = _zero_model(S.make_model(83, 1, 4, 4, [True, True], 1, 3, prune=None, prior=True))
    want = [[], []]
    for li, lv in enumerate(model["levels"]):
        hd = lv["prior"]
        ly = hd["layer"]
        ly["w"][:] = 0
        cb, px = ly["c_out"] // 2, lv["h"] * lv["w"]
        ly["bias"][:] = [1000 * (li + 1) + 97 * c for c in range(cb)] + [40 * (li + 1) + 55 * c for c in range(cb)]
        ly["s"][:] = 3
        hd["ls_lo"], hd["ls_hi"] = 0, 63
        vals = [_rq_exact(int(b), int(m), 3) for b, m in zip(ly["bias"], ly["m0"])]
        for c in range(cb):
            want[0] += [vals[c]] * px
            want[1] += [_clip(vals[cb + c], 0, 63)] * px
    x = S.smooth_field_images(84, 3, 4, 4, 1.0)[:, :1]
    _, p = O.forward(O.Packed(model), x)
    d, d_fact, _ = S.latent_sizes(model)
    assert p.shape == (3, 2, d_fact) and d_fact == len(want[0]) == 12
    for b in range(3):
        assert p[b, 0].tolist() == want[0]
        assert p[b, 1].tolist() == want[1]
    assert len(set(want[0])) == 6 and len(set(want[1])) > 2    # the blocks are distinguishable
