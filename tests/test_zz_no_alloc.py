"""The workspace-free entry point `salad_linear_attn_fwd_noalloc` against the regular one.

Some hosts of the library cannot hand it scratch memory at call time (an inference server with
a memory pool fixed at start-up, code that runs around CUDA-graph capture, a real-time loop that
must stay out of the driver's allocator).  For them the scratch is a fixed array inside the
library.  Because every call shares that array and it keeps the previous call's contents, the
check runs two calls in a row on different inputs and sizes: the second must not be disturbed
by what the first left behind.  This file sorts last on purpose, so that a failure here cannot
hide the result of any other test in a run that stops at the first failure."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

MAX_ABS = 2e-2
REL_L2 = 1e-2


def bf16_randn(shape, seed):
    rng = np.random.default_rng(seed)
    return torch.from_numpy(rng.standard_normal(shape).astype(np.float32)).to(torch.bfloat16).cuda()


def close(a, b, what):
    a = a.float().cpu().numpy().astype(np.float64)
    b = b.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(a).all(), what
    max_abs = np.abs(a - b).max()
    rel = np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-30)
    assert max_abs <= MAX_ABS and rel <= REL_L2, f"{what}: max_abs {max_abs:.3g} rel_l2 {rel:.3g}"


def test_noalloc_matches_workspace_entry_point_twice_in_a_row():
    from oracle import salad_oracle as orc
    from paper_2601_16515_b200 import salad

    # first call: 2 x 4 heads of 128 channels, ragged length; second call: other sizes, other data; third
    # call: the largest problem the fixed array holds (16 heads of 128 channels)
    for call, (B, H, N, d) in enumerate([(2, 4, 3000, 128), (1, 3, 1100, 64), (2, 8, 2000, 128)]):
        q, k, v = (bf16_randn((B, H, N, d), 10 * call + j) for j in range(3))
        ref_kv = torch.empty((B, H, d, d), dtype=torch.float32, device="cuda")
        ref_z = torch.empty((B, H, d), dtype=torch.float32, device="cuda")
        ref = salad.salad_linear_attn_fwd(q, k, v, eps=1e-6, kv_out=ref_kv, z_out=ref_z)

        out = torch.full_like(q, float("nan"))
        kv = torch.empty_like(ref_kv)
        z = torch.empty_like(ref_z)
        status = torch.ones(1, dtype=torch.int32, device="cuda")
        torch.cuda.synchronize()
        allocations = torch.cuda.memory_stats()["allocation.all.allocated"]     # running count of allocations made
        got = salad.salad_linear_attn_fwd_noalloc(q, k, v, eps=1e-6, out=out, kv_out=kv, z_out=z, status=status)
        torch.cuda.synchronize()
        # with `out` passed in, the binding asks torch's allocator for nothing either
        assert torch.cuda.memory_stats()["allocation.all.allocated"] == allocations
        assert int(status.item()) == 0
        assert got.data_ptr() == out.data_ptr()
        close(got, ref, f"call {call}: output")
        # ... and against the CPU oracle (Eq. 3), like every other entry point
        want = torch.from_numpy(orc.linear_attn(q.float().cpu().numpy(), k.float().cpu().numpy(),
                                                v.float().cpu().numpy(), eps=1e-6)).reshape(B, H, N, d)
        close(got, want, f"call {call}: output against the oracle")
        np.testing.assert_allclose(z.cpu().numpy(), ref_z.cpu().numpy(), rtol=1e-4, atol=1e-3)
        np.testing.assert_allclose(kv.cpu().numpy(), ref_kv.cpu().numpy(), rtol=1e-3,
                                   atol=float(ref_kv.abs().max()) * 1e-4)


def test_noalloc_rejects_sizes_beyond_its_fixed_scratch():
    from paper_2601_16515_b200 import salad

    B, H, N, d = 1, salad.NOALLOC_MAX_HEADS + 1, 256, 64
    q, k, v = (bf16_randn((B, H, N, d), j) for j in range(3))
    with pytest.raises(salad.SaladError) as err:
        salad.salad_linear_attn_fwd_noalloc(q, k, v)
    assert err.value.code == salad.SALAD_ERR_UNSUPPORTED
