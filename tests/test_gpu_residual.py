"""Couplings with the paper's residual-block network (Eq. 3, scatter add of Sec. 4.5) on the GPU
against the CPU oracle, bit for bit, through the C ABI: encode, decode, prior parameters and the
level-stepped decode."""
import numpy as np
import pytest

import iodf_synth as S
import oracle as O

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def G():
    import paper_2206_08869_b200 as g
    g.load_library()
    return g


def _t(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _both_ways(G, model, x, plan=0):
    import torch
    z_ref, p_ref = O.forward(O.Packed(model), x)
    m = G.iodf_create(model, x.shape[0], plan=plan)
    z, p = G.iodf_forward(m, _t(x))
    G.iodf_check(m)
    np.testing.assert_array_equal(z.cpu().numpy(), z_ref)
    if p_ref is not None:
        np.testing.assert_array_equal(p.cpu().numpy(), p_ref)
    oor = torch.zeros(1, dtype=torch.int32, device="cuda")
    p2 = torch.empty_like(p) if p is not None else None
    xr = G.iodf_inverse(m, _t(z_ref), prior=p2, out_of_range=oor)
    G.iodf_check(m)
    np.testing.assert_array_equal(xr.cpu().numpy(), x)
    assert int(oor.item()) == 0
    if p is not None:
        assert torch.equal(p, p2)
    return m, z_ref, p_ref


@pytest.mark.parametrize("hw,splits,couplings,hidden,blocks,prune,batch", [
    (8, [True], 1, 16, 1, None, 2),                       # 16 pixels, one block, nothing pruned
    (16, [True, True], 2, 24, 2, (0.4, 0.8), 5),          # 64- and 16-pixel levels, odd kept widths
    (32, [True, True, True], 2, 40, 2, (0.4, 0.7), 3),    # 256 pixels: two tiles per image
    (16, [True, False], 1, 128, 8, (0.4, 0.7), 2),        # the paper's width and depth: 128 channels, 8 blocks
    (64, [True, True], 1, 24, 2, (0.4, 0.7), 3),          # 1024 pixels: four row bands per image (a cluster), then 256
    (48, [True], 2, 16, 1, None, 2),                      # 576 pixels: four bands of six rows, image rows of 24 pixels
])
def test_residual_models_bit_exact(G, hw, splits, couplings, hidden, blocks, prune, batch):
    model = S.make_residual_model(0xE500 + hw + hidden, 3, hw, hw, splits, couplings, hidden, blocks, prune=prune)
    x = S.smooth_field_images(0xE600 + hw, batch, hw, hw, 2.0)
    _both_ways(G, model, x)


@pytest.mark.parametrize("hw,splits,couplings,hidden,blocks,prune,batch", [
    (8, [True, True], 2, 24, 2, (0.4, 0.8), 11),          # 16- and 4-pixel levels: 3 and 8 images per CTA, ragged last CTAs
    (16, [True, True, False], 1, 40, 2, (0.4, 0.7), 7),   # 64 pixels (one image per CTA), then 16 and 4 pixels
    (8, [True], 1, 128, 8, (0.4, 0.7), 4),                # the paper's width and depth at 16 pixels: 3 + 1 images
    (64, [True, True, True, True], 1, 16, 1, None, 5),    # row bands first (one band per CTA), grouped images at the end
])
def test_residual_models_throughput_plan(G, hw, splits, couplings, hidden, blocks, prune, batch):
    """The throughput plan puts as many images' padded frames into a CTA's tile as it holds: same
    results, in both directions, with the prior parameters and a last CTA that is not full."""
    model = S.make_residual_model(0xEB00 + hw + hidden, 3, hw, hw, splits, couplings, hidden, blocks, prune=prune)
    x = S.smooth_field_images(0xEC00 + hw, batch, hw, hw, 2.0)
    _both_ways(G, model, x, plan=G.IODF_PLAN_THROUGHPUT)


def test_first_level_of_the_imagenet64_geometry_at_the_papers_width(G):
    """App. B.1 on 64 x 64 images: the first level has 32 x 32 pixels, which one CTA cannot hold; it
    runs as four row bands per image whose edge rows are exchanged after every conv. Width 128, eight
    blocks, one coupling per level to keep the oracle's time down; batch position must not matter."""
    import torch
    model = S.make_residual_model(0xEA00, 3, 64, 64, [True, True], 1, 128, 8, prune=(0.4, 0.7))
    x = S.smooth_field_images(0xEA01, 3, 64, 64, 4.0)
    m, z_ref, p_ref = _both_ways(G, model, x)
    z1, _ = G.iodf_forward(m, _t(x[2:3]))
    np.testing.assert_array_equal(z1.cpu().numpy()[0], z_ref[2])


def test_index_lists_in_any_order_and_chunks_without_a_filter(G):
    """Sec. 4.5: the kept outputs go back to the channels the index list names, whatever its order.
    Here every block's list is shuffled (its filters stay paired with their channels' positions in
    the list), and the first block of each coupling keeps nothing among channels 16..31, so a whole
    16-channel group of the block tensor only gets the shortcut."""
    model = S.make_residual_model(0xE800, 3, 16, 16, [True, True], 2, 48, 3, prune=(0.3, 0.6))
    rng = np.random.default_rng(0xE801)
    for lv in model["levels"]:
        for cp in lv["couplings"]:
            for b, rb in enumerate(cp["blocks"]):
                ly = cp["layers"][2 + 2 * b]
                keep = np.arange(len(rb["idx"]))
                if b == 0:
                    keep = keep[(rb["idx"] < 16) | (rb["idx"] >= 32)]
                keep = rng.permutation(keep)
                rb["idx"] = np.ascontiguousarray(rb["idx"][keep])
                for k in ("w", "bias", "m0", "s"):
                    ly[k] = np.ascontiguousarray(ly[k][keep])
                if ly.get("gate") is not None:
                    ly["gate"] = np.ascontiguousarray(ly["gate"][keep])
                ly["c_out"] = len(keep)
                assert len(keep) > 0 and not np.all(np.diff(rb["idx"]) > 0)
    x = S.smooth_field_images(0xE802, 3, 16, 16, 2.0)
    _both_ways(G, model, x)


def test_residual_and_plain_levels_in_one_model_and_stepped_decode(G):
    """A model whose first level uses residual couplings and whose second the three-conv couplings;
    decoded level by level with the blocks that are not decoded yet poisoned."""
    import torch
    res = S.make_residual_model(0xE700, 3, 16, 16, [True, True], 2, 32, 2, prune=(0.4, 0.7))
    plain = S.make_model(0xE701, 3, 16, 16, [True, True], 2, 24, prune=(0.4, 0.7))
    model = {"in_c": 3, "in_h": 16, "in_w": 16, "levels": [res["levels"][0], plain["levels"][1]]}
    x = S.smooth_field_images(0xE702, 4, 16, 16, 2.0)
    m, z_ref, p_ref = _both_ways(G, model, x)
    lay = G.iodf_get_layout(m)
    z = torch.full((4, int(lay.d)), 0x7A7A7A7A, dtype=torch.int32, device="cuda")
    zf = int(lay.z_final_off)
    z[:, zf:] = _t(z_ref[:, zf:])
    prior = torch.full((4, 2, int(lay.d_fact)), -1, dtype=torch.int32, device="cuda")
    xr = torch.zeros((4, 3, 16, 16), dtype=torch.uint8, device="cuda")
    for lv in (1, 0):
        G.iodf_inverse_level(m, lv, G.IODF_LEVEL_PRIOR, z, prior=prior)
        zo, n = int(lay.z_off[lv]), (int(lay.level_c[lv]) // 2) * int(lay.level_h[lv]) * int(lay.level_w[lv])
        z[:, zo:zo + n] = _t(z_ref[:, zo:zo + n])
        G.iodf_inverse_level(m, lv, G.IODF_LEVEL_COUPLINGS, z, x_u8=xr if lv == 0 else None)
    G.iodf_check(m)
    np.testing.assert_array_equal(prior.cpu().numpy(), p_ref)
    np.testing.assert_array_equal(xr.cpu().numpy(), x)


def test_stepped_decode_with_several_images_per_cta(G):
    """Throughput plan, residual couplings at 64 and 16 pixels (one and three images per CTA), decoded
    level by level (prior head and couplings as separate launches), five images: a ragged last CTA."""
    import torch
    model = S.make_residual_model(0xED00, 3, 16, 16, [True, True], 2, 32, 2, prune=(0.4, 0.7))
    x = S.smooth_field_images(0xED01, 5, 16, 16, 2.0)
    m, z_ref, p_ref = _both_ways(G, model, x, plan=G.IODF_PLAN_THROUGHPUT)
    lay = G.iodf_get_layout(m)
    z = torch.full((5, int(lay.d)), 0x7A7A7A7A, dtype=torch.int32, device="cuda")
    zf = int(lay.z_final_off)
    z[:, zf:] = _t(z_ref[:, zf:])
    prior = torch.full((5, 2, int(lay.d_fact)), -1, dtype=torch.int32, device="cuda")
    xr = torch.zeros((5, 3, 16, 16), dtype=torch.uint8, device="cuda")
    for lv in (1, 0):
        G.iodf_inverse_level(m, lv, G.IODF_LEVEL_PRIOR, z, prior=prior)
        zo, n = int(lay.z_off[lv]), (int(lay.level_c[lv]) // 2) * int(lay.level_h[lv]) * int(lay.level_w[lv])
        z[:, zo:zo + n] = _t(z_ref[:, zo:zo + n])
        G.iodf_inverse_level(m, lv, G.IODF_LEVEL_COUPLINGS, z, x_u8=xr if lv == 0 else None)
    G.iodf_check(m)
    np.testing.assert_array_equal(prior.cpu().numpy(), p_ref)
    np.testing.assert_array_equal(xr.cpu().numpy(), x)


def test_config_r32_throughput_plan_equals_the_default_plan(G):
    """Config R32 at the benchmark's batch with the plan its steps in flight use (the 4 x 4 level takes
    three images per CTA): the same latents and prior parameters as the default plan, exact round trip."""
    import torch
    model = S.config_model("R32")
    x = _t(S.config_images("R32"))
    m0 = G.iodf_create(model, x.shape[0])
    m1 = G.iodf_create(model, x.shape[0], plan=G.IODF_PLAN_THROUGHPUT)
    z0, p0 = G.iodf_forward(m0, x)
    z1, p1 = G.iodf_forward(m1, x)
    G.iodf_check(m0)
    G.iodf_check(m1)
    assert torch.equal(z0, z1) and torch.equal(p0, p1)
    xr = G.iodf_inverse(m1, z1)
    G.iodf_check(m1)
    assert torch.equal(xr, x)


def test_config_r32_in_the_benchmarks_launch_configuration(G):
    """The paper's network on the ImageNet32 geometry at the benchmark's batch of 64: the oracle
    checks sampled images (first, last, two in between), the round trip covers the whole batch."""
    import torch
    model = S.config_model("R32")
    x = S.config_images("R32")
    B = x.shape[0]
    idx = np.array([0, 21, 42, B - 1])
    z_ref, p_ref = O.forward(O.Packed(model), x[idx])
    m = G.iodf_create(model, B)
    z, p = G.iodf_forward(m, _t(x))
    G.iodf_check(m)
    np.testing.assert_array_equal(z.cpu().numpy()[idx], z_ref)
    np.testing.assert_array_equal(p.cpu().numpy()[idx], p_ref)
    xr = G.iodf_inverse(m, z)
    G.iodf_check(m)
    np.testing.assert_array_equal(xr.cpu().numpy(), x)
    # an image's result does not depend on the batch around it
    z1, _ = G.iodf_forward(m, _t(x[5:6]))
    assert torch.equal(z1[0], z[5])


def test_branch_output_near_the_int32_limit(G):
    """A block's second conv with shift 0, a multiplier just under one and biases as large as the
    accumulator bound allows: its requantised outputs reach +-(2^31 - 2), and adding the shortcut
    byte must still clip to 0..255 as the oracle's 64-bit sum does."""
    model = S.make_residual_model(0xE900, 3, 8, 8, [True], 1, 16, 2, prune=None)
    for cp in model["levels"][0]["couplings"]:
        ly = cp["layers"][2]                       # conv_b of the first block
        worst = np.abs(ly["w"].astype(np.int64)).reshape(ly["c_out"], -1).sum(axis=1) * 255
        big = (2 ** 31 - 1) - worst
        ly["bias"][:] = np.where(np.arange(ly["c_out"]) % 2 == 0, big, -big).astype(np.int32)
        ly["m0"][:] = 2 ** 31 - 1
        ly["s"][:] = 0
    x = S.smooth_field_images(0xE901, 2, 8, 8, 2.0)
    _both_ways(G, model, x)


def test_config_r64_in_the_benchmarks_launch_configuration(G):
    """The paper's network on the ImageNet64 geometry (Sec. 5, App. B.1) at the benchmark's batch: the
    oracle checks two sampled images, the round trip covers the whole batch."""
    model = S.config_model("R64")
    x = S.config_images("R64")
    B = x.shape[0]
    idx = np.array([0, B - 1])
    z_ref, p_ref = O.forward(O.Packed(model), x[idx])
    m = G.iodf_create(model, B)
    z, p = G.iodf_forward(m, _t(x))
    G.iodf_check(m)
    np.testing.assert_array_equal(z.cpu().numpy()[idx], z_ref)
    np.testing.assert_array_equal(p.cpu().numpy()[idx], p_ref)
    xr = G.iodf_inverse(m, z)
    G.iodf_check(m)
    np.testing.assert_array_equal(xr.cpu().numpy(), x)
