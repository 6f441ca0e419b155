"""Level-stepped decode and patch-based coding through the C ABI, against the CPU oracle.

Level-stepped decode (the decompressor's order: the prior of a level's factored-out block is a
function of the channels the level keeps, App. B.1 / Sec. 3): every latent block that the entropy
decoder would not have produced yet is filled with a poison value, so a step that read it would
give wrong prior parameters or a wrong image.

Patch-based coding (Sec. 5.3): cutting an image into patches is pure data movement, written here
with numpy reshapes; the oracle encodes the resulting batch."""
import numpy as np
import pytest

import iodf_synth as S
import oracle as O

pytestmark = pytest.mark.gpu

POISON = 0x7A7A7A7A
SENTINEL = -77777


@pytest.fixture(scope="module")
def G():
    import paper_2206_08869_b200 as g
    g.load_library()
    return g


def _t(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


@pytest.mark.parametrize("hw,splits,hidden,batch", [
    (32, [True, True, True], 48, 5),      # 256-, 64- and 16-pixel levels, a prior head on each
    (16, [True, True, False], 40, 9),     # the last level keeps all its channels (no split, no prior)
    (64, [True, True], 64, 2),            # 1024-pixel first level: eight tiles per image
])
def test_level_stepped_decode_reads_only_what_is_decoded(G, hw, splits, hidden, batch):
    import torch
    model = S.make_model(0x5700 + hw, 3, hw, hw, splits, 3, hidden, prune=(0.4, 0.7))
    x = S.smooth_field_images(0x5800 + hw, batch, hw, hw, 2.0)
    z_ref, p_ref = O.forward(O.Packed(model), x)
    m = G.iodf_create(model, batch)
    lay = G.iodf_get_layout(m)
    L = int(lay.n_levels)
    d, d_fact = int(lay.d), int(lay.d_fact)

    z = torch.full((batch, d), POISON, dtype=torch.int32, device="cuda")
    zf = int(lay.z_final_off)
    z[:, zf:] = _t(z_ref[:, zf:])                       # the final block is decoded first
    prior = torch.full((batch, 2, max(d_fact, 1)), SENTINEL, dtype=torch.int32, device="cuda")
    xr = torch.zeros((batch, 3, hw, hw), dtype=torch.uint8, device="cuda")
    oor = torch.zeros(1, dtype=torch.int32, device="cuda")
    done = np.zeros(max(d_fact, 1), dtype=bool)         # prior entries emitted so far

    for lv in range(L - 1, -1, -1):
        c, h, w = int(lay.level_c[lv]), int(lay.level_h[lv]), int(lay.level_w[lv])
        n_out = (c // 2) * h * w if splits[lv] else 0
        if splits[lv]:
            po = int(lay.prior_off[lv])
            G.iodf_inverse_level(m, lv, G.IODF_LEVEL_PRIOR, z, prior=prior)
            G.iodf_check(m)
            got = prior.cpu().numpy()
            np.testing.assert_array_equal(got[:, :, po:po + n_out], p_ref[:, :, po:po + n_out])
            done[po:po + n_out] = True
            assert np.all(got[:, :, ~done] == SENTINEL)  # nothing but this level's entries was written
            zo = int(lay.z_off[lv])
            z[:, zo:zo + n_out] = _t(z_ref[:, zo:zo + n_out])   # "entropy-decode" the level's block
        else:
            with pytest.raises(G.IodfError):             # no prior head at this level
                G.iodf_inverse_level(m, lv, G.IODF_LEVEL_PRIOR, z, prior=prior)
        G.iodf_inverse_level(m, lv, G.IODF_LEVEL_COUPLINGS, z, x_u8=xr if lv == 0 else None, out_of_range=oor)
        G.iodf_check(m)
    np.testing.assert_array_equal(xr.cpu().numpy(), x)
    assert int(oor.item()) == 0
    if d_fact:
        np.testing.assert_array_equal(prior.cpu().numpy(), p_ref)
    # the one-call decode gives the same image
    assert torch.equal(G.iodf_inverse(m, _t(z_ref)), xr)


def _cut(image, ph, pw):
    """[C,H,W] -> [B,C,ph,pw], patches in row-major order."""
    C, H, W = image.shape
    return np.ascontiguousarray(image.reshape(C, H // ph, ph, W // pw, pw).transpose(1, 3, 0, 2, 4)
                                .reshape(-1, C, ph, pw))


@pytest.mark.parametrize("hw,splits,hidden,H,W", [
    (32, [True, True], 48, 96, 128),      # 12 patches, one image per CTA at the first level
    (8, [True], 24, 16, 40),              # 10 patches of 8x8: eight images share a CTA, ragged last group
    (64, [True, True, True, True], 32, 128, 192),   # 6 patches of the 64x64 flow
])
def test_patch_coding_equals_the_batch_of_cut_patches(G, hw, splits, hidden, H, W):
    import torch
    model = S.make_model(0x9A00 + hw, 3, hw, hw, splits, 2, hidden, prune=(0.4, 0.7))
    image = S.smooth_field_images(0x9B00 + hw, 1, H, W, 3.0)[0]          # [3,H,W]
    xb = _cut(image, hw, hw)
    B = xb.shape[0]
    z_ref, p_ref = O.forward(O.Packed(model), xb)
    m = G.iodf_create(model, B)
    z, p = G.iodf_forward_patches(m, _t(image))
    G.iodf_check(m)
    np.testing.assert_array_equal(z.cpu().numpy(), z_ref)
    np.testing.assert_array_equal(p.cpu().numpy(), p_ref)
    oor = torch.zeros(1, dtype=torch.int32, device="cuda")
    back = G.iodf_inverse_patches(m, z, H, W, out_of_range=oor)
    G.iodf_check(m)
    np.testing.assert_array_equal(back.cpu().numpy(), image)
    assert int(oor.item()) == 0
    # the plain batch entry point on the cut patches agrees
    z2, _ = G.iodf_forward(m, _t(xb))
    assert torch.equal(z, z2)


def test_patch_coding_of_residual_couplings_with_several_patches_per_cta(G):
    """Throughput plan, residual couplings on 4 x 4 patches (2 x 2 pixels at the first level: eight
    patches' padded frames share a CTA's tile), an image of 11 patches: the patch grid's index map,
    the grouped frames and a ragged last CTA together."""
    import torch
    model = S.make_residual_model(0x9D00, 3, 4, 4, [True], 2, 24, 2, prune=(0.4, 0.7))
    image = S.smooth_field_images(0x9D01, 1, 4, 44, 3.0)[0]
    xb = _cut(image, 4, 4)
    z_ref, p_ref = O.forward(O.Packed(model), xb)
    m = G.iodf_create(model, xb.shape[0], plan=G.IODF_PLAN_THROUGHPUT)
    z, p = G.iodf_forward_patches(m, _t(image))
    G.iodf_check(m)
    np.testing.assert_array_equal(z.cpu().numpy(), z_ref)
    np.testing.assert_array_equal(p.cpu().numpy(), p_ref)
    back = G.iodf_inverse_patches(m, z, 4, 44)
    G.iodf_check(m)
    np.testing.assert_array_equal(back.cpu().numpy(), image)


def test_patch_argument_errors(G):
    model = S.make_model(0x9C00, 3, 8, 8, [True], 1, 16)
    m = G.iodf_create(model, 4)
    import torch
    img = torch.zeros((3, 16, 20), dtype=torch.uint8, device="cuda")     # 20 is not a multiple of 8
    with pytest.raises(G.IodfError) as e:
        G.iodf_forward_patches(m, img)
    assert e.value.status == -1
    img = torch.zeros((3, 16, 24), dtype=torch.uint8, device="cuda")     # 6 patches > max_batch 4
    with pytest.raises(G.IodfError) as e:
        G.iodf_forward_patches(m, img)
    assert e.value.status == -1
