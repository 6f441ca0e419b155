"""iodf_forward_static: the encode for callers that must not allocate.

A plug-in living inside a host process that owns the device memory pool, or a service that meets a
batch larger than the max_batch its model was created for at a moment when allocating is off
limits, cannot use the workspace that iodf_create obtained with cudaMalloc. This entry point keeps
the data passed between the level kernels in a fixed array inside the library image instead. The
test calls it through the C ABI twice in a row and requires the same bits as iodf_forward and as
the CPU oracle; it runs last so that a run that stops at the first failure has already covered
everything else."""
import numpy as np
import pytest

import iodf_synth as S
import oracle as O

pytestmark = pytest.mark.gpu


def test_static_scratch_encode_matches_iodf_forward_twice():
    import torch
    import paper_2206_08869_b200 as G

    model = S.make_model(0x57A7, 3, 32, 32, [True, True, True], 3, 48, prune=(0.4, 0.7))
    big = G.iodf_create(model, 24)          # reference: ordinary entry point, allocated workspace
    small = G.iodf_create(model, 2)         # same model created for a tiny max_batch
    per_image = G.iodf_static_scratch_bytes_per_image(small)
    assert 0 < per_image * 24 <= G.IODF_STATIC_SCRATCH_BYTES

    for call, seed in enumerate((1, 2)):    # two calls in a row; the array keeps the first call's data
        x_host = S.smooth_field_images(seed, 24 - 5 * call, 32, 32, 2.0)
        x = torch.from_numpy(x_host).cuda()
        B = x.shape[0]
        z_ref, p_ref = G.iodf_forward(big, x)
        G.iodf_check(big)
        z = torch.full((B, small.d), -1, dtype=torch.int32, device="cuda")
        p = torch.full((B, 2, small.d_fact), -1, dtype=torch.int32, device="cuda")
        G.iodf_forward_static(small, x, z, p)   # B exceeds small's max_batch: allowed here
        G.iodf_check(small)
        assert torch.equal(z, z_ref), "call %d: latents differ" % call
        assert torch.equal(p, p_ref), "call %d: prior parameters differ" % call
        z_cpu, p_cpu = O.forward(O.Packed(model), x_host)      # and the expected bits themselves
        np.testing.assert_array_equal(z.cpu().numpy(), z_cpu)
        np.testing.assert_array_equal(p.cpu().numpy(), p_cpu)

    # beyond the fixed array: a clear error, nothing launched
    too_many = G.IODF_STATIC_SCRATCH_BYTES // per_image + 1
    x = torch.zeros((too_many, 3, 32, 32), dtype=torch.uint8, device="cuda")
    z = torch.empty((too_many, small.d), dtype=torch.int32, device="cuda")
    with pytest.raises(G.IodfError) as e:
        G.iodf_forward_static(small, x, z, None)
    assert e.value.status == -8
    assert "fixed capacity" in str(e.value)
