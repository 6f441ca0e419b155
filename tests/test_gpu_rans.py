"""GPU entropy coder against the CPU oracle: the coded words of every stream must be identical
(integer coding, so the bar is bit equality), the decoder must give z back, and the whole
decompressor (final block, then per level: prior parameters, entropy decode of the block, inverse
couplings) must recover the images from the coded words alone."""
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


def _valid(words, counts):
    """Zero everything past each stream's count (the container's tail is unspecified)."""
    w = words.copy()
    idx = np.arange(w.shape[2])[None, None, :]
    w[idx >= counts[:, :, None]] = 0
    return w


@pytest.mark.parametrize("hw,splits,hidden,batch,eps", [
    (32, [True, True, True], 32, 5, 256),
    (16, [True, True, False], 24, 9, 100),      # a last level without a split, ragged streams
    (64, [True, True, True, True], 24, 3, 256), # the ImageNet64 block structure
])
def test_coded_words_equal_the_oracles_and_decode(G, hw, splits, hidden, batch, eps):
    import torch
    model = S.make_model(0xAA00 + hw, 3, hw, hw, splits, 2, hidden, prune=(0.4, 0.7))
    codec = S.logistic_codec(elems_per_stream=eps)
    x = S.smooth_field_images(0xAB00 + hw, batch, hw, hw, 2.0)
    z_ref, p_ref = O.forward(O.Packed(model), x)
    w_ref, c_ref = O.rans_encode(codec, model, z_ref, p_ref)

    m = G.iodf_create(model, batch)
    cd = G.iodf_codec_create(m, codec)
    assert cd.n_streams == w_ref.shape[1] and cd.words_per_stream == w_ref.shape[2]
    z, p = G.iodf_forward(m, _t(x))
    words, counts = G.iodf_rans_encode(cd, z, p)
    G.iodf_codec_check(cd)
    wc = words.cpu().numpy().view(np.uint16)
    cc = counts.cpu().numpy().view(np.uint32)
    np.testing.assert_array_equal(cc, c_ref)
    np.testing.assert_array_equal(_valid(wc, cc), _valid(w_ref, c_ref))

    # decompressor: from the coded words alone
    lay = G.iodf_get_layout(m)
    zd = torch.full_like(z, 0x7A7A7A7A)
    pd = torch.full_like(p, -77777)
    xr = torch.zeros((batch, 3, hw, hw), dtype=torch.uint8, device="cuda")
    nb = cd.n_blocks
    G.iodf_rans_decode_block(cd, nb - 1, words, counts, pd, zd)           # the final block: fixed prior
    block_of_level = {int(cd.layout.block_level[q]): q for q in range(nb - 1)}
    for lv in range(int(lay.n_levels) - 1, -1, -1):
        if lv in block_of_level:
            G.iodf_inverse_level(m, lv, G.IODF_LEVEL_PRIOR, zd, prior=pd)
            G.iodf_rans_decode_block(cd, block_of_level[lv], words, counts, pd, zd)
        G.iodf_inverse_level(m, lv, G.IODF_LEVEL_COUPLINGS, zd, x_u8=xr if lv == 0 else None)
    G.iodf_check(m)
    G.iodf_codec_check(cd)
    np.testing.assert_array_equal(zd.cpu().numpy(), z_ref)
    np.testing.assert_array_equal(xr.cpu().numpy(), x)


def test_escapes_and_extreme_values(G):
    """Random int32 latents: nearly every element is an escape; the window's edge values and the
    ends of the int32 range are planted."""
    import torch
    model = S.make_model(0xAC00, 3, 16, 16, [True, True], 1, 16)
    codec = S.logistic_codec(elems_per_stream=64)
    rng = np.random.default_rng(5)
    B, d = 4, 3 * 16 * 16
    d_fact = 6 * 64 + 12 * 16
    z = rng.integers(-2**31, 2**31, (B, d)).astype(np.int32)
    prior = np.stack([rng.integers(-3000, 3000, (B, d_fact)), rng.integers(0, 64, (B, d_fact))], axis=1).astype(np.int32)
    z[0, :8] = prior[0, 0, :8] + np.array([2047, 2048, -2047, -2048, 0, 1, -1, 2049])
    z[1, :4] = [2**31 - 1, -2**31, 0, 0]
    w_ref, c_ref = O.rans_encode(codec, model, z, prior)
    m = G.iodf_create(model, B)
    cd = G.iodf_codec_create(m, codec)
    words, counts = G.iodf_rans_encode(cd, _t(z), _t(prior))
    G.iodf_codec_check(cd)
    cc = counts.cpu().numpy().view(np.uint32)
    np.testing.assert_array_equal(cc, c_ref)
    np.testing.assert_array_equal(_valid(words.cpu().numpy().view(np.uint16), cc), _valid(w_ref, c_ref))
    out = torch.zeros((B, d), dtype=torch.int32, device="cuda")
    for q in range(cd.n_blocks):
        G.iodf_rans_decode_block(cd, q, words, counts, _t(prior), out)
    G.iodf_codec_check(cd)
    np.testing.assert_array_equal(out.cpu().numpy(), z)


def test_model_without_prior_heads(G):
    """Every block then has the fixed prior (mu = 0, one scale index); no prior buffer is passed."""
    import torch
    model = S.make_model(0xAE00, 3, 16, 16, [True, True], 2, 16, prior=False)
    codec = S.logistic_codec(elems_per_stream=50, final_ls=50)
    x = S.smooth_field_images(0xAE01, 3, 16, 16, 2.0)
    z_ref, p_ref = O.forward(O.Packed(model), x)
    assert p_ref is None
    w_ref, c_ref = O.rans_encode(codec, model, z_ref, None)
    m = G.iodf_create(model, 3)
    cd = G.iodf_codec_create(m, codec)
    z, p = G.iodf_forward(m, _t(x))
    assert p is None
    words, counts = G.iodf_rans_encode(cd, z, None)
    G.iodf_codec_check(cd)
    cc = counts.cpu().numpy().view(np.uint32)
    np.testing.assert_array_equal(cc, c_ref)
    np.testing.assert_array_equal(_valid(words.cpu().numpy().view(np.uint16), cc), _valid(w_ref, c_ref))
    out = torch.zeros_like(z)
    for q in range(cd.n_blocks):
        G.iodf_rans_decode_block(cd, q, words, counts, None, out)
    G.iodf_codec_check(cd)
    assert torch.equal(out, z)


def test_bad_scale_index_and_damaged_stream_are_reported(G):
    import torch
    model = S.make_model(0xAD00, 3, 8, 8, [True], 1, 8)
    codec = S.logistic_codec(elems_per_stream=32)
    m = G.iodf_create(model, 2)
    cd = G.iodf_codec_create(m, codec)
    d, d_fact = 3 * 64, 6 * 16
    z = torch.zeros((2, d), dtype=torch.int32, device="cuda")
    prior = torch.zeros((2, 2, d_fact), dtype=torch.int32, device="cuda")
    prior[1, 1, 3] = 64                                   # one past the table
    words, counts = G.iodf_rans_encode(cd, z, prior)
    with pytest.raises(G.IodfError) as e:
        G.iodf_codec_check(cd)
    assert e.value.status == -9
    prior[1, 1, 3] = 0
    words, counts = G.iodf_rans_encode(cd, z, prior)
    G.iodf_codec_check(cd)
    counts[0, 0] -= 1                                     # a truncated stream
    out = torch.zeros_like(z)
    G.iodf_rans_decode_block(cd, 0, words, counts, prior, out)
    with pytest.raises(G.IodfError):
        G.iodf_codec_check(cd)
    # descriptor errors are caught on the host
    bad = dict(codec, final_ls=64)
    with pytest.raises(G.IodfError) as e:
        G.iodf_codec_create(m, bad)
    assert e.value.status == -1


def _packed_reference(words, counts):
    """The compact byte stream written out with numpy: offsets, then per image counts and words."""
    B, S, _ = words.shape
    recs = []
    for b in range(B):
        parts = [counts[b].astype("<u2").tobytes()]
        parts += [words[b, s, :counts[b, s]].astype("<u2").tobytes() for s in range(S)]
        recs.append(b"".join(parts))
    off = np.zeros(B + 1, dtype="<u4")
    off[1:] = np.cumsum([len(r) for r in recs])
    return off.tobytes() + b"".join(recs)


@pytest.mark.parametrize("hw,splits,batch,eps", [(32, [True, True, True], 7, 256), (16, [True, False], 33, 40)])
def test_compact_stream_and_host_round_trip(G, hw, splits, batch, eps):
    import torch
    model = S.make_model(0xAF00 + hw, 3, hw, hw, splits, 2, 24, prune=(0.4, 0.7))
    codec = S.logistic_codec(elems_per_stream=eps)
    x = S.smooth_field_images(0xAF10 + hw, batch, hw, hw, 2.0)
    z_ref, p_ref = O.forward(O.Packed(model), x)
    w_ref, c_ref = O.rans_encode(codec, model, z_ref, p_ref)
    want = _packed_reference(w_ref, c_ref)

    m = G.iodf_create(model, batch + 3)
    cd = G.iodf_codec_create(m, codec)
    z, p = G.iodf_forward(m, _t(x))
    words, counts = G.iodf_rans_encode(cd, z, p)
    packed, n = G.iodf_rans_pack(cd, words, counts)
    assert n == len(want) and n <= G.iodf_rans_packed_capacity(cd, batch)
    assert packed[:n].cpu().numpy().tobytes() == want
    w2, c2 = G.iodf_rans_unpack(cd, packed, n, batch)
    G.iodf_codec_check(cd)
    assert torch.equal(c2, counts)
    cc = counts.cpu().numpy().view(np.uint32)
    np.testing.assert_array_equal(_valid(w2.cpu().numpy().view(np.uint16), cc), _valid(w_ref, c_ref))

    # images -> bytes -> images through the host-buffer calls
    xh = torch.from_numpy(x).pin_memory()
    out, nb = G.iodf_compress_host(m, cd, xh)
    assert out[:nb].numpy().tobytes() == want
    back = G.iodf_decompress_host(m, cd, out, nb, batch)
    torch.cuda.synchronize()
    G.iodf_check(m)
    G.iodf_codec_check(cd)
    np.testing.assert_array_equal(back.numpy(), x)
    # a byte stream cut short is reported, not read past its end
    G.iodf_decompress_host(m, cd, out, nb - 10, batch)
    with pytest.raises(G.IodfError):
        G.iodf_codec_check(cd)
    with pytest.raises(G.IodfError):                          # too small an output buffer
        G.iodf_compress_host(m, cd, xh, out_host=torch.empty(64, dtype=torch.uint8).pin_memory())
