"""CUDA path vs CPU oracle, element by element, through the C ABI. Everything is integer, so the
bar is bit-exact equality of z, the prior parameters and the reconstructed x."""
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


def _check_both_ways(G, model, x, max_batch=None, sample=None, plan=0):
    """Encode x on the GPU and compare with the oracle (all images, or the `sample` indices);
    decode the oracle's z on the GPU and compare with x."""
    import torch
    B = x.shape[0]
    pk = O.Packed(model)
    idx = np.arange(B) if sample is None else np.asarray(sample)
    z_ref, p_ref = O.forward(pk, x[idx])
    m = G.iodf_create(model, max_batch or B, plan=plan)
    z, p = G.iodf_forward(m, _t(x))
    G.iodf_check(m)
    zc = z.cpu().numpy()
    np.testing.assert_array_equal(zc[idx], z_ref)
    if p_ref is not None:
        np.testing.assert_array_equal(p.cpu().numpy()[idx], p_ref)
    # decode what the GPU encoded (full batch): exact round trip, and the same prior parameters
    oor = torch.zeros(1, dtype=torch.int32, device="cuda")
    p2 = torch.empty_like(p) if p is not None else None
    xr = G.iodf_inverse(m, z, prior=p2, out_of_range=oor)
    G.iodf_check(m)
    np.testing.assert_array_equal(xr.cpu().numpy(), x)
    assert int(oor.item()) == 0
    if p is not None:
        assert torch.equal(p, p2)
    return m, zc


# ---- small shapes: several tiles, ragged tails, odd widths ---------------------------------------
@pytest.mark.parametrize("hw,splits,hidden,prune,batch", [
    (8, [False], 16, None, 3),                   # 16 px per image: several images share one tile
    (8, [True, True], 24, (0.4, 0.7), 5),        # ragged last group (5 images, 8 and 32 per CTA)
    (16, [True, True, True], 40, (0.4, 0.7), 9), # three levels, odd kept widths
    (12, [True, False], 20, (0.4, 0.7), 7),      # 36-px and 9-px levels: tiles straddle images
    (4, [True], 8, None, 70),                    # 4-px level: 32 images per CTA, three CTAs
    (32, [True, True], 64, (0.4, 0.7), 3),       # 256-px level: two tiles per image
    (16, [True, True], 320, None, 5),            # hidden width above 256: weights streamed in K-slices
    (8, [True], 500, (0.6, 1.0), 3),             # odd widths between 300 and 500
])
def test_small_models_bit_exact(G, hw, splits, hidden, prune, batch):
    model = S.make_model(100 + hw, 3, hw, hw, splits, 3, hidden, prune=prune)
    x = S.smooth_field_images(200 + hw, batch, hw, hw, 1.5)
    _check_both_ways(G, model, x)


def test_adversarial_inputs_and_wraparound(G):
    import torch
    model = S.make_model(7, 3, 16, 16, [True, True], 4, 32, prune=(0.4, 0.7))
    x = np.concatenate([np.zeros((1, 3, 16, 16), np.uint8), np.full((1, 3, 16, 16), 255, np.uint8),
                        S.Stream(8, "u8").integers(0, 256, 2 * 3 * 256).astype(np.uint8).reshape(2, 3, 16, 16)])
    m, _ = _check_both_ways(G, model, x)
    # any int32 vector is a latent: decode must agree with the oracle, including values far outside 0..255
    pk = O.Packed(model)
    zr = S.Stream(9, "z").integers(-(1 << 31), 1 << 31, 4 * pk.d).astype(np.int32).reshape(4, pk.d)
    xu_ref, xi_ref, p_ref, oor_ref = O.inverse(pk, zr)
    oor = torch.zeros(1, dtype=torch.int32, device="cuda")
    p = torch.empty((4, 2, pk.d_fact), dtype=torch.int32, device="cuda")
    xu = G.iodf_inverse(m, _t(zr), prior=p, out_of_range=oor)
    G.iodf_check(m)
    np.testing.assert_array_equal(xu.cpu().numpy(), xu_ref)
    np.testing.assert_array_equal(p.cpu().numpy(), p_ref)
    assert int(oor.item()) == oor_ref and oor_ref > 0


def test_zero_shift_layers_take_the_exact_path(G):
    """s = 0 in a hidden layer (multiplier in [1/2, 1)) must match as well."""
    model = S.make_model(17, 3, 8, 8, [True], 2, 12, prune=None)
    for cp in model["levels"][0]["couplings"]:
        cp["layers"][0]["s"][:] = 0
        cp["layers"][1]["s"][::2] = 0
        cp["in_s"] = 0
    x = S.smooth_field_images(18, 4, 8, 8, 1.0)
    _check_both_ways(G, model, x)


def test_biases_around_the_folding_limit(G):
    """The library folds a hidden layer's biases into spare rows of its GEMM while every |bias| is at
    most 63 + 7 * 127 * 127 = 112966 and adds them in the epilogue otherwise; both routes, the exact
    limit on either side, and layers that mix small and extreme biases must agree with the oracle.
    (Per-channel shifts that differ within a layer take yet another route.)"""
    limit = 63 + 7 * 127 * 127
    model = S.make_model(23, 3, 16, 16, [True, True], 4, 48, prune=(0.5, 0.8))
    edge = [limit, -limit, limit - 1, 1 - limit, 127 * 127, -127 * 127, 64, -64, 63, -63, 0]
    for lv in model["levels"]:
        for ci, cp in enumerate(lv["couplings"]):
            for li in range(2):
                ly = cp["layers"][li]
                n = len(ly["bias"])
                if ci == 0:      # all foldable, every edge value present
                    ly["bias"][:len(edge)] = edge[:n]
                elif ci == 1:    # one channel just past the limit: the whole layer adds in the epilogue
                    ly["bias"][:len(edge)] = edge[:n]
                    ly["bias"][n // 2] = limit + 1 if li == 0 else -(limit + 1)
                elif ci == 2:    # large biases
                    ly["bias"][::3] = 1 << 20
                    ly["bias"][1::3] = -(1 << 20)
                else:            # foldable biases, but shifts differ inside the layer
                    ly["bias"][:len(edge)] = edge[:n]
                    ly["s"][::2] += 1
    x = S.smooth_field_images(24, 6, 16, 16, 1.5)
    _check_both_ways(G, model, x)


def test_unsigned_hidden_activations(G):
    """Hidden activations in the unsigned 8-bit format (0..255 after the ReLU, Sec. 4.1): the next
    conv then reads an unsigned A operand. Shifts are lowered by two so that a good share of the
    activations lies in 128..255 and some saturate at 255; couplings mix the formats (both layers
    unsigned; only the first; a clip at 200; unsigned with biases too large to fold; unsigned with
    per-channel shifts)."""
    model = S.make_model(29, 3, 32, 32, [True, True, True], 5, 56, prune=(0.5, 0.9), act_hi=255)
    for lv in model["levels"]:
        for ci, cp in enumerate(lv["couplings"]):
            for li in range(2):
                ly = cp["layers"][li]
                ly["s"][:] = np.maximum(ly["s"] - 2, 1)
            if ci == 1:
                cp["layers"][1]["clamp"] = (0, 127)
                cp["layers"][1]["s"][:] += 2
            elif ci == 2:
                cp["layers"][0]["clamp"] = (0, 200)
                cp["layers"][1]["clamp"] = (3, 255)
            elif ci == 3:
                cp["layers"][0]["bias"][::2] = 1 << 20
                cp["layers"][1]["bias"][1::2] = -(1 << 19)
            elif ci == 4:
                cp["layers"][0]["s"][::2] += 1
    x = S.smooth_field_images(30, 6, 32, 32, 2.0)
    # activations above 127 must really occur and matter: clipping at 127 instead changes z
    import copy
    narrow = copy.deepcopy(model)
    for lv in narrow["levels"]:
        for cp in lv["couplings"]:
            for li in range(2):
                lo, hi = cp["layers"][li]["clamp"]
                cp["layers"][li]["clamp"] = (lo, min(hi, 127))
    assert not np.array_equal(O.forward(O.Packed(model), x[:1])[0], O.forward(O.Packed(narrow), x[:1])[0])
    _check_both_ways(G, model, x)


def test_zero_bias_and_no_prior(G):
    model = S.make_model(19, 3, 16, 16, [True, False], 2, 16, prune=None, prior=False, with_bias=False)
    _check_both_ways(G, model, S.smooth_field_images(20, 4, 16, 16, 1.5))


def test_batch_limits_and_argument_errors(G):
    import torch
    model = S.make_model(21, 3, 8, 8, [True], 1, 8, prune=None)
    m = G.iodf_create(model, 4)
    x = _t(S.smooth_field_images(22, 5, 8, 8, 1.0))
    with pytest.raises(G.IodfError) as e:
        G.iodf_forward(m, x)                     # batch 5 > max_batch 4
    assert e.value.status == -1
    z = torch.empty((4, m.d + 1), dtype=torch.int32, device="cuda").reshape(-1)[1:1 + 4 * m.d].reshape(4, m.d)
    with pytest.raises(G.IodfError) as e:
        G.iodf_forward(m, x[:4].contiguous(), z=z)   # z not 16-byte aligned
    assert e.value.status == -1
    z1, _ = G.iodf_forward(m, x[:1].contiguous())    # batch 1
    z4, _ = G.iodf_forward(m, x[:4].contiguous())
    G.iodf_check(m)
    assert torch.equal(z1[0], z4[0])


def test_repeat_runs_are_identical(G):
    import torch
    model = S.config_model(0)
    m = G.iodf_create(model, 16)
    x = _t(S.config_images(0))
    z1, _ = G.iodf_forward(m, x)
    z2, _ = G.iodf_forward(m, x)
    G.iodf_check(m)
    assert torch.equal(z1, z2)


def test_host_buffer_entry_points(G):
    import torch
    model = S.make_model(23, 3, 16, 16, [True, True], 2, 24, prune=(0.4, 0.7))
    x = S.smooth_field_images(24, 6, 16, 16, 1.5)
    z_ref, p_ref = O.forward(O.Packed(model), x)
    m = G.iodf_create(model, 8)
    hx = torch.from_numpy(x).pin_memory()
    hz = torch.empty((6, m.d), dtype=torch.int32).pin_memory()
    hp = torch.empty((6, 2, m.d_fact), dtype=torch.int32).pin_memory()
    G.iodf_forward_host(m, hx, hz, hp)
    G.iodf_check(m)
    np.testing.assert_array_equal(hz.numpy(), z_ref)
    np.testing.assert_array_equal(hp.numpy(), p_ref)
    hx2 = torch.empty_like(hx)
    G.iodf_inverse_host(m, hz, hx2)
    G.iodf_check(m)
    np.testing.assert_array_equal(hx2.numpy(), x)


# ---- the five benchmark configurations ------------------------------------------------------------
# ---- the throughput plan: as many images per CTA as a tile holds -----------------------------------
@pytest.mark.parametrize("hw,splits,hidden,prune,batch", [
    (8, [True, True], 24, (0.4, 0.7), 21),       # 16- and 4-px levels: 8 and 32 images per CTA, ragged last CTAs
    (16, [True, True, True], 40, (0.4, 0.7), 37),# 64-, 16- and 4-px levels
    (12, [True, False], 20, (0.4, 0.7), 50),     # 36- and 9-px levels: images that do not divide the tile
    (16, [True, True], 320, None, 9),            # hidden width above 256: streamed weights only at one image per CTA
])
def test_throughput_plan_small_models_bit_exact(G, hw, splits, hidden, prune, batch):
    model = S.make_model(300 + hw, 3, hw, hw, splits, 3, hidden, prune=prune)
    x = S.smooth_field_images(400 + hw, batch, hw, hw, 1.5)
    _check_both_ways(G, model, x, plan=G.IODF_PLAN_THROUGHPUT)


def test_plans_differ_in_images_per_cta_as_documented(G):
    """Config 2 at batch 128: one image per CTA at every level under the default plan; under the
    throughput plan two at the 64-pixel level and four at the 16-pixel level (a full tile there would
    need streamed weights). Config R32: three 4 x 4 images' padded frames per tile."""
    model = S.config_model(2)
    m0, m1 = G.iodf_create(model, 128), G.iodf_create(model, 128, plan=G.IODF_PLAN_THROUGHPUT)
    assert [G.iodf_level_images_per_cta(m0, lv) for lv in range(4)] == [1, 1, 1, 1]
    assert [G.iodf_level_images_per_cta(m1, lv) for lv in range(4)] == [1, 1, 2, 4]
    r = S.config_model("R32")
    r0, r1 = G.iodf_create(r, 64), G.iodf_create(r, 64, plan=G.IODF_PLAN_THROUGHPUT)
    assert [G.iodf_level_images_per_cta(r0, lv) for lv in range(3)] == [1, 1, 1]
    assert [G.iodf_level_images_per_cta(r1, lv) for lv in range(3)] == [1, 1, 3]
    with pytest.raises(G.IodfError):
        G.iodf_level_images_per_cta(m0, 4)


def test_throughput_plan_config2_equals_the_latency_plan(G):
    """The benchmark keeps several batches in flight on handles made with the throughput plan: same
    latents and prior parameters as the oracle on sampled images, as the default plan on all, exact
    round trip, and three handles running at the same time on three streams give the same again."""
    import torch
    x = S.config_images(2)
    B = x.shape[0]
    pick = sorted(set([0, 1, B // 2, B - 1] + S.Stream(6, "pick").integers(0, B, 8).tolist()))
    model = S.config_model(2)
    m, z = _check_both_ways(G, model, x, sample=pick, plan=G.IODF_PLAN_THROUGHPUT)
    m0 = G.iodf_create(model, B)
    z0, p0 = G.iodf_forward(m0, _t(x))
    G.iodf_check(m0)
    np.testing.assert_array_equal(z0.cpu().numpy(), z)
    lanes = [(m, torch.cuda.Stream())] + [(G.iodf_create(model, B, plan=G.IODF_PLAN_THROUGHPUT), torch.cuda.Stream())
                                          for _ in range(2)]
    xs = [_t(np.ascontiguousarray(np.roll(x, k, axis=0))) for k in range(3)]
    outs = [(torch.empty_like(z0), torch.empty_like(p0)) for _ in lanes]      # a lane's own buffers, reused
    torch.cuda.synchronize()
    for rep in range(4):
        for k, (mk, st) in enumerate(lanes):
            G.iodf_forward(mk, xs[k], outs[k][0], outs[k][1], stream=st)
    torch.cuda.synchronize()
    for k, (mk, _) in enumerate(lanes):
        G.iodf_check(mk)
        np.testing.assert_array_equal(outs[k][0].cpu().numpy(), np.roll(z, k, axis=0))
        assert torch.equal(outs[k][1], torch.roll(p0, k, dims=0))


def test_config0_tiny_flow(G):
    _check_both_ways(G, S.config_model(0), S.config_images(0))


def test_config1_imagenet32_encode_full_batch(G):
    _check_both_ways(G, S.config_model(1), S.config_images(1))


def test_config2_imagenet64_encode(G):
    """Full batch of 128 in the launch configuration the benchmark times; the oracle checks a
    sample (first, last, group boundaries, seeded random picks); the remaining images are covered
    by the exact round trip and by batch independence."""
    import torch
    x = S.config_images(2)
    B = x.shape[0]
    pick = sorted(set([0, 1, B // 2 - 1, B // 2, B - 2, B - 1] + S.Stream(5, "pick").integers(0, B, 10).tolist()))
    m, z = _check_both_ways(G, S.config_model(2), x, sample=pick)
    z8, _ = G.iodf_forward(m, _t(x[40:48]))
    G.iodf_check(m)
    np.testing.assert_array_equal(z8.cpu().numpy(), z[40:48])


def test_config3_decode_of_config1(G):
    import torch
    model, x = S.config_model(3), S.config_images(3)
    pk = O.Packed(model)
    z_ref, p_ref = O.forward(pk, x)
    m = G.iodf_create(model, x.shape[0])
    p = torch.empty((x.shape[0], 2, pk.d_fact), dtype=torch.int32, device="cuda")
    xr = G.iodf_inverse(m, _t(z_ref), prior=p)
    G.iodf_check(m)
    np.testing.assert_array_equal(xr.cpu().numpy(), x)
    np.testing.assert_array_equal(p.cpu().numpy(), p_ref)


@pytest.mark.parametrize("batch", [1, 8, 64, 512, 2048])
def test_config4_batch_sweep_pruned(G, batch):
    """Encode and decode at each batch size. The oracle checks up to 12 sampled images; beyond
    batch 64 the GPU result must also equal the concatenation of batch-64 runs."""
    import torch
    model = S.config_model(4)
    x = S.config_images(4, batch=batch)
    pick = sorted(set([0, batch - 1] + S.Stream(batch, "pick").integers(0, batch, 10).tolist()))
    m, z = _check_both_ways(G, model, x, sample=pick)
    if batch > 64:
        for b0 in range(0, batch, 64):
            z64, _ = G.iodf_forward(m, _t(x[b0:b0 + 64]))
            np.testing.assert_array_equal(z64.cpu().numpy(), z[b0:b0 + 64])
        G.iodf_check(m)


@pytest.mark.parametrize("batch", [1, 8, 64, 512, 2048])
def test_config4_batch_sweep_stress_width_512(G, batch):
    """The unpruned width-512 variant of the ImageNet64-shaped flow (weights streamed from L2 per
    tile). The oracle checks up to 6 sampled images per batch size."""
    model = S.config_model("4s")
    x = S.config_images("4s", batch=batch)
    pick = sorted(set([0, batch - 1] + S.Stream(batch, "pick512").integers(0, batch, 4).tolist()))
    m, z = _check_both_ways(G, model, x, sample=pick)
    if batch > 64:
        for b0 in range(0, batch, 64):
            z64, _ = G.iodf_forward(m, _t(x[b0:b0 + 64]))
            np.testing.assert_array_equal(z64.cpu().numpy(), z[b0:b0 + 64])
        G.iodf_check(m)


@pytest.mark.parametrize("hw,hidden,prune,batch", [
    (64, 40, (0.4, 0.7), 3),     # 1024-pixel first level: eight tiles, per-tap partials in columns of their own
    (48, 24, None, 2),           # 576 pixels: five tiles, a ragged last one, image rows that straddle warps
    (64, 200, None, 2),          # wide hidden layers: the per-tap partials share the slot's columns
])
def test_levels_of_many_tiles_in_the_role_split_kernel(G, hw, hidden, prune, batch):
    """First levels of four tiles and more run in the kernel that gives the im2col / shifted sum,
    the requantisation and the MMA issue to different warps; the deeper levels of the same models
    run in the general kernel. Encode, prior parameters, decode and the out-of-range count against
    the oracle, for every image."""
    model = S.make_model(0xB100 + hw + hidden, 3, hw, hw, [True, True], 3, hidden, prune=prune)
    x = S.smooth_field_images(0xB200 + hw, batch, hw, hw, 3.0)
    _check_both_ways(G, model, x)
