"""GPU parity of the linear branch with a rotary position embedding (Sec. 4.1) against the CPU
oracle, through the C ABI binding: the state, the linear-only call and the fused call."""
import numpy as np
import pytest
import torch

from oracle import salad_oracle as orc
from paper_2601_16515_b200 import workloads as wlmod
from test_gpu_parity import assert_close, dev_csr, f32, rand_qkv, random_csr, status_ok, stratified_rows

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def salad():
    from paper_2601_16515_b200 import salad as s
    return s


def random_table(N, d, seed):
    ang = np.random.default_rng(seed).uniform(-np.pi, np.pi, size=(N, d // 2))
    return np.stack([np.cos(ang), np.sin(ang)], axis=-1).astype(np.float16)     # the library's table dtype


@pytest.mark.parametrize("B,H,N,d", [(1, 2, 1024, 64), (2, 3, 1000, 128), (1, 1, 70, 128), (1, 2, 5000, 64),
                                     (1, 13, 3000, 128)])
def test_linear_rope(salad, B, H, N, d):
    q, k, v = rand_qkv(B, H, N, d, 900 + N)
    rope = random_table(N, d, N)
    kv = torch.empty((B, H, d, d), dtype=torch.float32, device="cuda")
    z = torch.empty((B, H, d), dtype=torch.float32, device="cuda")
    status = torch.ones(1, dtype=torch.int32, device="cuda")
    out = salad.salad_linear_attn_rope_fwd(q.cuda(), k.cuda(), v.cuda(), torch.from_numpy(rope).cuda(),
                                           eps=1e-6, kv_out=kv, z_out=z, status=status)
    status_ok(status)
    kv_ref, z_ref = orc.linear_state_rope(f32(k), f32(v), rope)
    np.testing.assert_allclose(z.cpu().numpy(), z_ref, rtol=1e-4, atol=1e-3)
    # the rotated keys are rounded to bf16 before the tensor cores (2^-9 relative per term, independent
    # over the N terms of an entry): the state matches to a few 1e-3 of its norm
    kv_g = kv.cpu().numpy().astype(np.float64)
    assert np.linalg.norm(kv_g - kv_ref) <= 5e-3 * np.linalg.norm(kv_ref)
    assert np.abs(kv_g - kv_ref).max() <= 1e-2 * np.abs(kv_ref).max()
    ref = orc.linear_attn_rope(f32(q), f32(k), f32(v), rope, eps=1e-6)
    assert_close(f32(out.cpu()).reshape(-1, d), ref, "linear rope")


def test_linear_rope_with_zero_angles_is_the_plain_branch(salad):
    B, H, N, d = 1, 3, 2000, 128
    q, k, v = rand_qkv(B, H, N, d, 77)
    ident = np.zeros((N, d // 2, 2), np.float16); ident[..., 0] = 1.0
    kv_a = torch.empty((B, H, d, d), dtype=torch.float32, device="cuda"); kv_b = torch.empty_like(kv_a)
    a = salad.salad_linear_attn_rope_fwd(q.cuda(), k.cuda(), v.cuda(), torch.from_numpy(ident).cuda(), kv_out=kv_a)
    b = salad.salad_linear_attn_fwd(q.cuda(), k.cuda(), v.cuda(), kv_out=kv_b)
    assert torch.equal(kv_a, kv_b)          # a rotation by zero is exact, the products are the same
    assert_close(f32(a.cpu()), f32(b.cpu()), "zero angles")


@pytest.mark.parametrize("B,H,N,d,Bq,Hm", [(1, 2, 1000, 128, 128, 2), (2, 2, 777, 64, 64, 1), (1, 3, 1300, 128, 64, 3),
                                           (2, 2, 900, 64, 128, 4)])
def test_fused_rope_small_shapes(salad, B, H, N, d, Bq, Hm):
    wl = wlmod.Workload("t", B, H, d, (1, 1, N), Bq, 64, (), 1)
    q, k, v = rand_qkv(B, H, N, d, 500 + N)
    rope = random_table(N, d, 3 * N)
    rp, ci = random_csr(Hm * wl.nQb, wl.nKb, 23 + N, lo=0, hi=min(wl.nKb, 9))
    rng = np.random.default_rng(N)
    lam = rng.uniform(0, 1, H).astype(np.float32); s = rng.uniform(0, 1, B).astype(np.float32)
    rp_d, ci_d = dev_csr(rp, ci)
    status = torch.ones(1, dtype=torch.int32, device="cuda")
    out = salad.salad_fused_rope_fwd(q.cuda(), k.cuda(), v.cuda(), rp_d, ci_d, Hm, torch.from_numpy(lam).cuda(),
                                     torch.from_numpy(s).cuda(), torch.from_numpy(rope).cuda(), Bq=Bq, status=status)
    status_ok(status)
    ref = orc.salad_fused_rope(f32(q), f32(k), f32(v), rope, Bq, 64, rp, ci, Hm, lam, s)
    assert_close(f32(out.cpu()).reshape(-1, d), ref, "fused rope small")


def test_fused_rope_tiny_config_with_the_3d_table(salad):
    wl = wlmod.C1
    q, k, v = wlmod.make_qkv(wl)
    T, Hs, Ws = wl.grid
    rp, ci = orc.mask_build(T, Hs, Ws, wl.Bq, wl.Bk, wl.windows)
    lam, s = wlmod.make_scales(wl)
    rope = orc.rope3d_table_vectorized(wl.grid, wl.d)
    rp_d, ci_d = dev_csr(rp, ci)
    args = (q.cuda(), k.cuda(), v.cuda(), rp_d, ci_d, wl.Hm, torch.from_numpy(lam).cuda(), torch.from_numpy(s).cuda(),
            torch.from_numpy(rope).cuda())
    status = torch.ones(1, dtype=torch.int32, device="cuda")
    out = salad.salad_fused_rope_fwd(*args, Bq=wl.Bq, status=status)
    status_ok(status)
    ref = orc.salad_fused_rope(f32(q), f32(k), f32(v), rope, wl.Bq, wl.Bk, rp, ci, wl.Hm, lam, s)
    assert_close(f32(out.cpu()).reshape(-1, wl.d), ref, "fused rope tiny")
    # a threshold above every scale drops the branch: the sparse output bit for bit
    dropped = salad.salad_fused_rope_fwd(*args, Bq=wl.Bq, drop_tau=2.0)
    sparse = salad.salad_sparse_attn_fwd(q.cuda(), k.cuda(), v.cuda(), rp_d, ci_d, wl.Hm, Bq=wl.Bq)
    assert torch.equal(dropped, sparse)
    # and it differs from the call without the table
    plain = salad.salad_fused_fwd(*args[:-1], Bq=wl.Bq)
    assert (out.float() - plain.float()).abs().max() > 1e-2


def test_fused_rope_wan13b_90_sampled(salad):
    wl = wlmod.C2
    q, k, v = wlmod.make_qkv(wl)
    T, Hs, Ws = wl.grid
    lam, s = wlmod.make_scales(wl)
    rope = orc.rope3d_table_vectorized(wl.grid, wl.d)
    rp_d, ci_d = salad.salad_mask_build(T, Hs, Ws, wl.Bq, wl.Bk, wl.windows)
    rp, ci = rp_d.cpu().numpy(), ci_d.cpu().numpy()
    status = torch.ones(1, dtype=torch.int32, device="cuda")
    out = salad.salad_fused_rope_fwd(q.cuda(), k.cuda(), v.cuda(), rp_d, ci_d, 1, torch.from_numpy(lam).cuda(),
                                     torch.from_numpy(s).cuda(), torch.from_numpy(rope).cuda(), Bq=wl.Bq,
                                     status=status).cpu()
    status_ok(status)
    sel = stratified_rows(wl, rp, 1)                     # every head; four of them with a row in every query block
    ref = orc.salad_fused_rope(f32(q), f32(k), f32(v), rope, wl.Bq, wl.Bk, rp, ci, 1, lam, s, sel=sel)
    got = f32(out).reshape(-1, wl.d)[sel]
    assert_close(got, ref, "fused rope wan1.3b-90", tight=True)


def test_rope_argument_checks(salad):
    B, H, N, d = 1, 1, 256, 64
    q, k, v = (t.cuda() for t in rand_qkv(B, H, N, d, 5))
    good = torch.from_numpy(random_table(N, d, 1)).cuda()
    with pytest.raises(ValueError):
        salad.salad_linear_attn_rope_fwd(q, k, v, good[:, :-1].contiguous())
    with pytest.raises(ValueError):
        salad.salad_linear_attn_rope_fwd(q, k, v, good.float())
    with pytest.raises(ValueError):
        salad.salad_linear_attn_rope_fwd(q, k, v, good.cpu())


def test_fused_rope_drops_per_batch_item(salad):
    # two batch items, one scale below the threshold: its linear branch is skipped on the device
    B, H, N, d, Bq = 2, 2, 1100, 128, 128
    wl = wlmod.Workload("t", B, H, d, (1, 1, N), Bq, 64, (), 1)
    q, k, v = rand_qkv(B, H, N, d, 4242)
    rope = random_table(N, d, 8)
    rp, ci = random_csr(wl.nQb, wl.nKb, 31, lo=1, hi=6)
    lam = np.array([0.9, 0.4], np.float32); s = np.array([0.2, 0.8], np.float32)
    rp_d, ci_d = dev_csr(rp, ci)
    status = torch.ones(1, dtype=torch.int32, device="cuda")
    out = salad.salad_fused_rope_fwd(q.cuda(), k.cuda(), v.cuda(), rp_d, ci_d, 1, torch.from_numpy(lam).cuda(),
                                     torch.from_numpy(s).cuda(), torch.from_numpy(rope).cuda(), Bq=Bq, status=status,
                                     drop_tau=0.5)
    status_ok(status)
    ref = orc.salad_fused_rope(f32(q), f32(k), f32(v), rope, Bq, 64, rp, ci, 1, lam, s, tau=0.5)
    assert_close(f32(out.cpu()).reshape(-1, d), ref, "fused rope drop")
    sparse = salad.salad_sparse_attn_fwd(q.cuda(), k.cuda(), v.cuda(), rp_d, ci_d, 1, Bq=Bq)
    assert torch.equal(out[0], sparse[0]) and not torch.equal(out[1], sparse[1])


def test_fused_rope_call_in_a_cuda_graph_and_repeatable(salad):
    B, H, N, d = 1, 4, 2048, 128
    q, k, v = (t.cuda() for t in rand_qkv(B, H, N, d, 911))
    rope = torch.from_numpy(orc.rope3d_table_vectorized((4, 16, 32), d)).cuda()
    rp, ci = salad.salad_mask_build(4, 16, 32, 128, 64, [(1, 3, 8)])
    lam = torch.rand(H, device="cuda"); s = torch.rand(B, device="cuda")
    ws = salad.alloc_workspace(B, H, N, d)
    status = torch.ones(1, dtype=torch.int32, device="cuda")
    eager = salad.salad_fused_rope_fwd(q, k, v, rp, ci, 1, lam, s, rope, workspace=ws, status=status)
    again = salad.salad_fused_rope_fwd(q, k, v, rp, ci, 1, lam, s, rope, workspace=ws, status=status)
    torch.cuda.synchronize()
    assert torch.equal(eager, again)             # fixed summation orders: bit-identical from call to call
    out = torch.zeros_like(q)
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            salad.salad_fused_rope_fwd(q, k, v, rp, ci, 1, lam, s, rope, out=out, workspace=ws, status=status,
                                       stream=side)
    for _ in range(3):
        out.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert torch.equal(out, eager)


@pytest.mark.parametrize("grid,d", [((3, 4, 5), 32), ((4, 16, 16), 64), ((2, 7, 9), 128)])
def test_rope3d_table_bit_exact(salad, grid, d):
    got = salad.salad_rope3d_table_build(*grid, d).cpu().numpy()
    ref = orc.rope3d_table(grid, d)
    assert got.dtype == np.float16 and got.shape == ref.shape
    assert np.array_equal(got.view(np.uint16), ref.view(np.uint16))


def test_rope3d_table_wan13b_shape_sampled_and_feeds_the_fused_call(salad):
    wl = wlmod.C2
    table = salad.salad_rope3d_table_build(*wl.grid, wl.d)
    tok = np.random.default_rng(11).integers(0, wl.N, size=400)
    ref = orc.rope3d_table(wl.grid, wl.d, tokens=tok)
    assert np.array_equal(table.cpu().numpy()[tok].view(np.uint16), ref.view(np.uint16))
    # other bases and the argument checks
    t2 = salad.salad_rope3d_table_build(2, 3, 4, 64, base=500.0).cpu().numpy()
    assert np.array_equal(t2.view(np.uint16), orc.rope3d_table((2, 3, 4), 64, base=500.0).view(np.uint16))
    with pytest.raises(salad.SaladError):
        salad.salad_rope3d_table_build(2, 3, 4, 64, base=1.0)
    # the device-built table is the one the rotary calls take
    q, k, v = (t.cuda() for t in wlmod.make_qkv(wl, heads=[0, 1]))
    a = salad.salad_linear_attn_rope_fwd(q, k, v, table)
    b = salad.salad_linear_attn_rope_fwd(q, k, v, torch.from_numpy(orc.rope3d_table_vectorized(wl.grid, wl.d)).cuda())
    assert torch.equal(a, b)
