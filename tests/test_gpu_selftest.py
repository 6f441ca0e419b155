"""The library's failure path and its tensor-peak microbenchmark on the GPU, through the C ABI.

The bounded wait is made to run out in the permitted way: a one-warp kernel waits a few tries on a
barrier that nothing arrives on, sets the status word and returns; nothing faults, traps or hangs."""
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


def test_a_wait_that_runs_out_is_reported_once_and_the_model_still_works(G):
    import torch
    model = S.make_model(0x7100, 3, 16, 16, [True, True], 2, 24, prune=(0.4, 0.7))
    x = S.smooth_field_images(0x7101, 5, 16, 16, 2.0)
    z_ref, p_ref = O.forward(O.Packed(model), x)
    m = G.iodf_create(model, 8)
    xt = torch.from_numpy(x).cuda()
    z, p = G.iodf_forward(m, xt)
    G.iodf_check(m)                                   # clean before the probe
    G.iodf_selftest_timeout(m, tries=3)
    with pytest.raises(G.IodfError) as e:
        G.iodf_check(m)
    assert e.value.status == -5                       # IODF_ETIMEOUT
    assert "wait" in G.iodf_strerror(-5)
    G.iodf_check(m)                                   # the status word was cleared by the report
    z2, p2 = G.iodf_forward(m, xt)                    # the context and the model are intact
    G.iodf_check(m)
    np.testing.assert_array_equal(z2.cpu().numpy(), z_ref)
    np.testing.assert_array_equal(p2.cpu().numpy(), p_ref)
    xr = G.iodf_inverse(m, z2)
    G.iodf_check(m)
    np.testing.assert_array_equal(xr.cpu().numpy(), x)
    with pytest.raises(G.IodfError):
        G.iodf_selftest_timeout(m, tries=0)           # argument check: 1..100 tries


def test_int8_mma_microbenchmark_runs_and_is_plausible(G):
    import torch
    model = S.make_model(0x7102, 3, 8, 8, [False], 1, 8, prune=None, prior=False)
    m = G.iodf_create(model, 1)
    stream = torch.cuda.current_stream()
    ops = G.iodf_int8_mma_peak(m, 2000)               # warm-up
    assert ops == 2 * 128 * 256 * 32 * 8 * 2000 * torch.cuda.get_device_properties(0).multi_processor_count
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    ops = G.iodf_int8_mma_peak(m, 20000)
    e1.record(stream)
    e1.synchronize()
    G.iodf_check(m)
    tops = ops / (e0.elapsed_time(e1) * 1e-3) / 1e12
    # nominal dense int8 is 4 500 TOP/s; anything outside this window means the kernel is not doing
    # (only) the multiplies it claims
    assert 1000.0 < tops < 5000.0, tops
