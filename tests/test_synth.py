"""The input generator: determinism, shapes, pruning law and value ranges."""
import numpy as np

import iodf_synth as S


def test_streams_are_counter_based():
    a = S.Stream(1, "x").uniform(10)
    st = S.Stream(1, "x")
    b = np.concatenate([st.uniform(4), st.uniform(6)])
    np.testing.assert_array_equal(a, b)
    assert (S.Stream(1, "y").uniform(10) != a).any()
    p = S.Stream(3, "p").permutation(17)
    assert sorted(p.tolist()) == list(range(17))
    n = S.Stream(4, "n").normal(200000)
    assert abs(n.mean()) < 0.01 and abs(n.std() - 1.0) < 0.01


def test_images_follow_recipe():
    x = S.smooth_field_images(9, 8, 32, 32, 2.0)
    assert x.dtype == np.uint8 and x.shape == (8, 3, 32, 32)
    np.testing.assert_array_equal(x, S.smooth_field_images(9, 8, 32, 32, 2.0))
    assert 105 < x.mean() < 135 and 45 < x.std() < 70
    # smooth: neighbouring pixels correlate strongly
    f = x.astype(np.float64)
    c = np.corrcoef(f[..., :-1].ravel(), f[..., 1:].ravel())[0, 1]
    assert c > 0.8


def test_config_models():
    m0 = S.config_model(0)
    assert [(lv["c"], lv["h"], lv["w"]) for lv in m0["levels"]] == [(12, 16, 16)]
    assert len(m0["levels"][0]["couplings"]) == 4
    perms = [cp["perm"].tolist() for cp in m0["levels"][0]["couplings"]]
    assert perms[0] == list(range(12)) and perms[1] == list(range(11, -1, -1))
    assert S.model_macs(m0) == 11008 * 256 * 4
    m2 = S.config_model(2)
    assert [(lv["c"], lv["h"], lv["w"]) for lv in m2["levels"]] == [(12, 32, 32), (24, 16, 16), (48, 8, 8), (96, 4, 4)]
    widths = [ly["c_out"] for lv in m2["levels"] for cp in lv["couplings"] for ly in cp["layers"][:2]]
    assert all(w % 2 == 1 and 0.4 * 256 - 1 <= w <= 0.7 * 256 + 1 for w in widths)
    d, d_fact, blocks = S.latent_sizes(m2)
    assert d == 3 * 64 * 64 and d_fact == 6144 + 3072 + 1536 + 768
    for lv in m2["levels"]:
        for cp in lv["couplings"]:
            for ly in cp["layers"]:
                assert ly["w"].dtype == np.int8 and np.abs(ly["w"].astype(int)).max() <= 127
                assert (ly["m0"] >= 1 << 30).all() and (ly["s"] >= 0).all() and (ly["s"] <= 31).all()
