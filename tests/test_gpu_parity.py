"""GPU parity: every entry point of libsalad, called through the C ABI binding, against the
CPU oracle on the same seeded inputs.  Mask lists are compared bit for bit; bf16 outputs
within max-abs 2e-2 and relative-L2 1e-2 (the tolerance of the benchmark spec; the bf16
rounding of an O(1) output alone is up to 2^-9 relative, and P is rounded to bf16 before the
P V product)."""
import numpy as np
import pytest
import torch

from oracle import salad_oracle as orc
from paper_2601_16515_b200 import workloads as wlmod

pytestmark = pytest.mark.gpu

MAX_ABS = 2e-2
REL_L2 = 1e-2
# Regression bound for the Wan-shaped workloads, next to the contract bound above: the kernels deliver
# about 2e-3 / 2e-3 there (one bf16 rounding of an output of magnitude below one, bf16 P and state), so a
# several-fold loss of accuracy fails even though it would still be inside the contract.
TIGHT_MAX_ABS = 5e-3
TIGHT_REL_L2 = 4e-3


@pytest.fixture(scope="module")
def salad():
    from paper_2601_16515_b200 import salad as s
    return s


def assert_close(got, ref, what="", tight=False):
    got = np.asarray(got, dtype=np.float64); ref = np.asarray(ref, dtype=np.float64)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    max_abs = np.abs(got - ref).max()
    rel = np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30)
    assert max_abs <= MAX_ABS and rel <= REL_L2, f"{what}: max_abs {max_abs:.4g} rel_l2 {rel:.4g}"
    if tight:
        assert max_abs <= TIGHT_MAX_ABS and rel <= TIGHT_REL_L2, \
            f"{what}: inside the contract but worse than the regression bound: max_abs {max_abs:.4g} rel_l2 {rel:.4g}"
    return max_abs, rel


class Guarded:
    """A device tensor with a canary margin on each side: `t` is what the library gets, `check()` asserts
    that nothing outside it was written.  (compute-sanitizer is not available here; this is the stand-in for
    out-of-bounds writes around outputs and scratch.)"""
    MARGIN = 4096
    CANARY = 0xA5

    def __init__(self, shape, dtype, fill=None):
        n = int(np.prod(shape)) * torch.empty(0, dtype=dtype).element_size()
        self.n = n
        self.raw = torch.full((2 * self.MARGIN + n,), self.CANARY, dtype=torch.uint8, device="cuda")
        self.t = self.raw[self.MARGIN:self.MARGIN + n].view(dtype).view(*shape)
        if fill is not None:
            self.t.fill_(fill)

    def check(self, what=""):
        torch.cuda.synchronize()
        lo, hi = self.raw[:self.MARGIN], self.raw[self.MARGIN + self.n:]
        assert bool((lo == self.CANARY).all()) and bool((hi == self.CANARY).all()), f"{what}: write outside the buffer"


def status_ok(status):
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "kernel reported an expired wait"


def bf16(a):
    return torch.from_numpy(np.asarray(a, dtype=np.float32)).to(torch.bfloat16)


def rand_qkv(B, H, N, d, seed, scale=1.0):
    rng = np.random.default_rng(seed)
    return tuple(bf16(rng.standard_normal((B, H, N, d)) * scale) for _ in range(3))


def random_csr(rows, nKb, seed, lo=0, hi=None):
    rng = np.random.default_rng(seed)
    hi = nKb if hi is None else hi
    rp, cols = [0], []
    for _ in range(rows):
        row = np.sort(rng.choice(nKb, size=int(rng.integers(lo, hi + 1)), replace=False))
        cols.append(row); rp.append(rp[-1] + len(row))
    ci = np.concatenate(cols).astype(np.int32) if rp[-1] else np.zeros(0, np.int32)
    return np.asarray(rp, np.int32), ci


def dev_csr(rp, ci):
    ci_d = torch.from_numpy(ci if len(ci) else np.zeros(1, np.int32)).cuda()
    return torch.from_numpy(rp).cuda(), ci_d


def f32(t):
    return t.float().numpy()


# ------------------------------------------------------------------------------ mask builder

MASK_CASES = [
    ((2, 2, 4), 4, 4, [(0, 1, 0)]),
    ((3, 5, 7), 16, 8, [(1, 1, 2), (0, 0, 0), (3, 5, 7)]),
    ((4, 6, 6), 32, 16, [(0, 2, 2), (2, 0, 0)]),
    ((2, 9, 11), 64, 32, [(1, 3, 4)]),
    ((5, 3, 1), 4, 8, [(1, 1, 0)]),                       # Ws = 1: key blocks span many grid rows
    (wlmod.C1.grid, 64, 64, list(wlmod.C1.windows)),
    (wlmod.C1.grid, 64, 64, [(1, 1, 1), (0, 5, 5)]),
    (wlmod.C2.grid, 128, 64, [(2, 5, 24), (5, 5, 24), (1, 4, 24), (21, 30, 52), (0, 0, 0)]),
]


@pytest.mark.parametrize("grid,Bq,Bk,windows", MASK_CASES)
def test_mask_bit_exact(salad, grid, Bq, Bk, windows):
    T, Hs, Ws = grid
    rp, ci = salad.salad_mask_build(T, Hs, Ws, Bq, Bk, windows)
    rp_ref, ci_ref = orc.mask_build(T, Hs, Ws, Bq, Bk, windows)
    assert np.array_equal(rp.cpu().numpy(), rp_ref)
    assert np.array_equal(ci.cpu().numpy(), ci_ref)


def test_mask_bit_exact_wan14b_shape(salad):
    wl = wlmod.C4
    T, Hs, Ws = wl.grid
    rp, ci = salad.salad_mask_build(T, Hs, Ws, wl.Bq, wl.Bk, wl.windows)
    rp_ref, ci_ref = orc.mask_build(T, Hs, Ws, wl.Bq, wl.Bk, wl.windows)
    assert np.array_equal(rp.cpu().numpy(), rp_ref) and np.array_equal(ci.cpu().numpy(), ci_ref)
    sparsity = 1.0 - len(ci_ref) / (wl.nQb * wl.nKb)
    assert 0.89 < sparsity < 0.91


def test_mask_capacity_error(salad):
    import ctypes
    T, Hs, Ws = wlmod.C1.grid
    win = (ctypes.c_int32 * 3)(0, 15, 15)
    rp = torch.empty(17, dtype=torch.int32, device="cuda")
    ci = torch.full((8,), -7, dtype=torch.int32, device="cuda")
    nnz = ctypes.c_int64(0)
    rc = salad._lib.salad_mask_build(T, Hs, Ws, 64, 64, 1, win, ctypes.c_void_p(rp.data_ptr()),
                                     ctypes.c_void_p(ci.data_ptr()), 8, ctypes.byref(nnz), None)
    assert rc == salad.SALAD_ERR_CAPACITY and nnz.value == 64
    assert (ci.cpu() == -7).all()


# ------------------------------------------------------------------------------ sparse branch

SMALL_SHAPES = [
    # B, H, N, d, Bq, Hm
    (1, 2, 1024, 64, 64, 2),
    (1, 2, 1024, 128, 128, 1),
    (2, 3, 1000, 128, 128, 3),      # ragged: last q block 104 rows, last key block 40 keys
    (1, 2, 200, 64, 128, 1),        # N < 2 tiles, ragged
    (1, 1, 712, 64, 64, 1),         # odd number of 64-row query blocks (12), ragged
    (1, 2, 1100, 128, 64, 2),
]


@pytest.mark.parametrize("B,H,N,d,Bq,Hm", SMALL_SHAPES)
def test_sparse_random_lists(salad, B, H, N, d, Bq, Hm):
    q, k, v = rand_qkv(B, H, N, d, 100 + N)
    nQb, nKb = -(-N // Bq), -(-N // 64)
    rp, ci = random_csr(Hm * nQb, nKb, 7 + N, lo=0, hi=nKb)       # includes empty and full rows
    rp_d, ci_d = dev_csr(rp, ci)
    g_out, g_lse = Guarded((B, H, N, d), torch.bfloat16, fill=1.0), Guarded((B, H, N), torch.float32)
    g_ws = Guarded((salad.salad_workspace_bytes(B, H, N, d, Bq, 64),), torch.uint8)
    lse = g_lse.t
    status = torch.ones(1, dtype=torch.int32, device="cuda")
    out = salad.salad_sparse_attn_fwd(q.cuda(), k.cuda(), v.cuda(), rp_d, ci_d, Hm, Bq=Bq, out=g_out.t, lse=lse,
                                      workspace=g_ws.t, status=status)
    status_ok(status)
    for g, name in ((g_out, "out"), (g_lse, "lse"), (g_ws, "workspace")):
        g.check(f"sparse {name}")
    ref, ref_lse = orc.sparse_attn(f32(q), f32(k), f32(v), Bq, 64, rp, ci, Hm)
    assert_close(f32(out.cpu()).reshape(-1, d), ref, "sparse")
    got_lse = lse.cpu().numpy().reshape(-1)
    empty = np.isneginf(ref_lse)
    assert np.array_equal(np.isneginf(got_lse), empty)
    np.testing.assert_allclose(got_lse[~empty], ref_lse[~empty], atol=2e-3, rtol=1e-4)


def test_sparse_empty_rows_write_exact_zeros(salad):
    # Query blocks with no kept key block: Eq. 2 sums over nothing, the output row is exactly zero.
    # Half of the rows are empty, the others keep everything; repeated, on a buffer prefilled with
    # ones, so that a query tile landing in the staging buffer late would show up.
    B, H, N, d, Bq = 2, 3, 1000, 128, 128
    q, k, v = rand_qkv(B, H, N, d, 31)
    nQb, nKb = -(-N // Bq), -(-N // 64)
    lens = np.array([nKb if (r % 3 == 1) else 0 for r in range(H * nQb)], dtype=np.int32)
    rp = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    ci = np.concatenate([np.arange(n, dtype=np.int32) for n in lens if n] or [np.zeros(0, np.int32)])
    rp_d, ci_d = dev_csr(rp, ci)
    ref, _ = orc.sparse_attn(f32(q), f32(k), f32(v), Bq, 64, rp, ci, H)
    ref = ref.reshape(B, H, N, d)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    for _ in range(5):
        out = torch.ones_like(qd)
        salad.salad_sparse_attn_fwd(qd, kd, vd, rp_d, ci_d, H, Bq=Bq, out=out)
        got = f32(out.cpu()).reshape(B, H, N, d)
        for h in range(H):
            for i in range(nQb):
                if lens[h * nQb + i] == 0:
                    assert not got[:, h, i * Bq:(i + 1) * Bq].any(), (h, i)
        assert_close(got.reshape(-1, d), ref.reshape(-1, d), "half-empty")


def test_sparse_all_kept_is_full_attention(salad):
    B, H, N, d = 1, 2, 1000, 128
    q, k, v = rand_qkv(B, H, N, d, 5)
    rp, ci = wlmod.dense_csr(-(-N // 128), -(-N // 64), 1)
    rp_d, ci_d = dev_csr(rp, ci)
    out = salad.salad_sparse_attn_fwd(q.cuda(), k.cuda(), v.cuda(), rp_d, ci_d, 1)
    ref = torch.nn.functional.scaled_dot_product_attention(q.double(), k.double(), v.double())   # Eq. 1
    assert_close(f32(out.cpu()), ref.numpy(), "dense")


def test_sparse_softmax_scale_and_large_scores(salad):
    # scores with a wide dynamic range force the running-max rescale of the accumulator
    B, H, N, d = 1, 1, 1024, 128
    q, k, _ = rand_qkv(B, H, N, d, 6, scale=3.0)
    _, _, v = rand_qkv(B, H, N, d, 6, scale=1.0)       # outputs stay O(1): the tolerance is absolute
    rp, ci = wlmod.dense_csr(N // 128, N // 64, 1)
    rp_d, ci_d = dev_csr(rp, ci)
    for scale in (0.25, 1.0 / np.sqrt(d)):
        out = salad.salad_sparse_attn_fwd(q.cuda(), k.cuda(), v.cuda(), rp_d, ci_d, 1, softmax_scale=scale)
        ref, _ = orc.sparse_attn(f32(q), f32(k), f32(v), 128, 64, rp, ci, 1, scale=scale)
        assert_close(f32(out.cpu()).reshape(-1, d), ref, f"scale {scale}")


# ------------------------------------------------------------------------------ linear branch

@pytest.mark.parametrize("B,H,N,d", [(1, 2, 1024, 64), (2, 3, 1000, 128), (1, 1, 70, 128), (1, 2, 5000, 64)])
def test_linear(salad, B, H, N, d):
    q, k, v = rand_qkv(B, H, N, d, 200 + N)
    g_kv, g_z = Guarded((B, H, d, d), torch.float32), Guarded((B, H, d), torch.float32)
    g_out = Guarded((B, H, N, d), torch.bfloat16, fill=1.0)
    g_ws = Guarded((salad.salad_workspace_bytes(B, H, N, d, 128, 64),), torch.uint8)
    kv, z = g_kv.t, g_z.t
    status = torch.ones(1, dtype=torch.int32, device="cuda")
    out = salad.salad_linear_attn_fwd(q.cuda(), k.cuda(), v.cuda(), eps=1e-6, out=g_out.t, kv_out=kv, z_out=z,
                                      workspace=g_ws.t, status=status)
    status_ok(status)
    for g, name in ((g_out, "out"), (g_kv, "kv_out"), (g_z, "z_out"), (g_ws, "workspace")):
        g.check(f"linear {name}")
    kv_ref, z_ref = orc.linear_state(f32(k), f32(v))
    np.testing.assert_allclose(z.cpu().numpy(), z_ref, rtol=1e-4, atol=1e-3)
    np.testing.assert_allclose(kv.cpu().numpy(), kv_ref, rtol=1e-3, atol=np.abs(kv_ref).max() * 1e-4)
    ref = orc.linear_attn(f32(q), f32(k), f32(v), eps=1e-6)
    assert_close(f32(out.cpu()).reshape(-1, d), ref, "linear")


def test_linear_nonpositive_q_gives_zero(salad):
    B, H, N, d = 1, 1, 256, 64
    q, k, v = rand_qkv(B, H, N, d, 1)
    out = salad.salad_linear_attn_fwd((-q.abs()).cuda(), k.cuda(), v.cuda())
    assert (out == 0).all()
    # eps = 0: the rows with ReLU(Q_n) = 0 are 0/0, defined as 0 (not NaN), in the linear-only call and
    # in the fused call, where a NaN would also wipe out the sparse branch of the row
    qz = q.clone(); qz[:, :, ::3] = -qz[:, :, ::3].abs()
    out0 = salad.salad_linear_attn_fwd(qz.cuda(), k.cuda(), v.cuda(), eps=0.0)
    assert torch.isfinite(out0.float()).all() and (out0[:, :, ::3] == 0).all()
    assert_close(f32(out0.cpu()).reshape(-1, d), orc.linear_attn(f32(qz), f32(k), f32(v), eps=0.0), "eps = 0")
    rp, ci = wlmod.dense_csr(-(-N // 128), -(-N // 64), 1)
    rp_d, ci_d = dev_csr(rp, ci)
    one = torch.ones(1, device="cuda")
    fused0 = salad.salad_fused_fwd(qz.cuda(), k.cuda(), v.cuda(), rp_d, ci_d, 1, one, one, eps=0.0)
    ref = orc.salad_fused(f32(qz), f32(k), f32(v), 128, 64, rp, ci, 1, np.ones(1), np.ones(1), eps=0.0)
    assert_close(f32(fused0.cpu()).reshape(-1, d), ref, "fused, eps = 0")


# ------------------------------------------------------------------------------ fused

def run_fused(salad, wl, q, k, v, rp, ci, Hm, lam, s, guard=False, **kw):
    rp_d, ci_d = dev_csr(rp, ci)
    status = torch.ones(1, dtype=torch.int32, device="cuda")
    guards = []
    if guard:       # canary margins around the output and the scratch memory
        B, H, N, d = q.shape
        guards = [Guarded((B, H, N, d), torch.bfloat16, fill=1.0),
                  Guarded((salad.salad_workspace_bytes(B, H, N, d, wl.Bq, wl.Bk),), torch.uint8)]
        kw = dict(kw, out=guards[0].t, workspace=guards[1].t)
    out = salad.salad_fused_fwd(q.cuda(), k.cuda(), v.cuda(), rp_d, ci_d, Hm,
                                torch.from_numpy(lam).cuda(), torch.from_numpy(s).cuda(),
                                Bq=wl.Bq, Bk=wl.Bk, status=status, **kw)
    status_ok(status)
    for g in guards:
        g.check("fused call")
    return out


def test_fused_tiny_config_full(salad):
    wl = wlmod.C1
    q, k, v = wlmod.make_qkv(wl)
    T, Hs, Ws = wl.grid
    rp_d, ci_d = salad.salad_mask_build(T, Hs, Ws, wl.Bq, wl.Bk, wl.windows)
    rp, ci = orc.mask_build(T, Hs, Ws, wl.Bq, wl.Bk, wl.windows)
    assert np.array_equal(rp_d.cpu().numpy(), rp) and np.array_equal(ci_d.cpu().numpy(), ci)
    lam, s = wlmod.make_scales(wl)
    out = run_fused(salad, wl, q, k, v, rp, ci, wl.Hm, lam, s)
    ref = orc.salad_fused(f32(q), f32(k), f32(v), wl.Bq, wl.Bk, rp, ci, wl.Hm, lam, s)
    assert_close(f32(out.cpu()).reshape(-1, wl.d), ref, "fused tiny")


@pytest.mark.parametrize("B,H,N,d,Bq,Hm", SMALL_SHAPES)
def test_fused_small_shapes(salad, B, H, N, d, Bq, Hm):
    wl = wlmod.Workload("t", B, H, d, (1, 1, N), Bq, 64, (), 1)
    q, k, v = rand_qkv(B, H, N, d, 300 + N)
    rp, ci = random_csr(Hm * wl.nQb, wl.nKb, 17 + N, lo=0, hi=min(wl.nKb, 9))
    rng = np.random.default_rng(N)
    lam = rng.uniform(0, 1, H).astype(np.float32); s = rng.uniform(0, 1, B).astype(np.float32)
    out = run_fused(salad, wl, q, k, v, rp, ci, Hm, lam, s, guard=True)
    ref = orc.salad_fused(f32(q), f32(k), f32(v), Bq, 64, rp, ci, Hm, lam, s)
    assert_close(f32(out.cpu()).reshape(-1, d), ref, "fused small")


def test_fused_zero_scale_is_sparse_bit_for_bit(salad):
    wl = wlmod.C1
    q, k, v = wlmod.make_qkv(wl)
    T, Hs, Ws = wl.grid
    rp, ci = orc.mask_build(T, Hs, Ws, wl.Bq, wl.Bk, wl.windows)
    lam, s = wlmod.make_scales(wl)
    fused0 = run_fused(salad, wl, q, k, v, rp, ci, wl.Hm, np.zeros_like(lam), s)
    rp_d, ci_d = dev_csr(rp, ci)
    sparse = salad.salad_sparse_attn_fwd(q.cuda(), k.cuda(), v.cuda(), rp_d, ci_d, wl.Hm, Bq=wl.Bq)
    assert torch.equal(fused0, sparse)
    # and the fused result equals sparse + scale * linear computed by the standalone calls
    fused = run_fused(salad, wl, q, k, v, rp, ci, wl.Hm, lam, s)
    lin = salad.salad_linear_attn_fwd(q.cuda(), k.cuda(), v.cuda())
    c = torch.from_numpy(s)[:, None] * torch.from_numpy(lam)[None, :]
    comb = sparse.float().cpu() + c[:, :, None, None] * lin.float().cpu()
    assert_close(f32(fused.cpu()), comb.numpy(), "fused vs parts")


def stratified_rows(wl, rp, Hm, dense_heads=4, seed=0):
    """Output rows (flat index (b*H + h)*N + n) for a sampled check of a full-size run, chosen from the
    lists so that no kind of work item goes unseen: for EVERY (batch, head) the query blocks with the
    longest and the shortest kept list, the first block and the (ragged) last block, each with its first
    row, its last valid row and a random one; and for `dense_heads` (batch, head) pairs spread over the
    batch one random row in every query block."""
    rng = np.random.default_rng([wl.seed, 555, seed])
    B, H, N, Bq, nQb = wl.B, wl.H, wl.N, wl.Bq, wl.nQb
    BH = B * H
    rows = []
    dense = set(np.unique(np.linspace(0, BH - 1, min(dense_heads, BH)).round().astype(int)).tolist())
    for bh in range(BH):
        h = bh % H
        hm = 0 if Hm == 1 else (h if Hm == H else bh)
        lens = np.diff(rp[hm * nQb:(hm + 1) * nQb + 1])
        blocks = {0, nQb - 1, int(np.argmax(lens)), int(np.argmin(lens))}
        if bh in dense:
            blocks |= set(range(nQb))
        for i in blocks:
            n0, n1 = i * Bq, min(N, (i + 1) * Bq)
            picks = [int(rng.integers(n0, n1))] if (bh in dense and i not in (0, nQb - 1)) else \
                    [n0, n1 - 1, int(rng.integers(n0, n1))]
            rows += [bh * N + n for n in picks]
    return np.unique(np.asarray(rows, dtype=np.int64))


def fused_check(salad, wl, full=False, windows=None, csr=None, dense_heads=4):
    """Full-size run on the GPU in the configuration the benchmark times, against the oracle on the
    same tensors: the whole output (full=True) or a stratified sample of its rows over all heads."""
    q, k, v = wlmod.make_qkv(wl)
    T, Hs, Ws = wl.grid
    lam, s = wlmod.make_scales(wl)
    if csr is None:
        windows = wl.windows if windows is None else windows
        rp_d, ci_d = salad.salad_mask_build(T, Hs, Ws, wl.Bq, wl.Bk, windows)
        rp, ci = orc.mask_build(T, Hs, Ws, wl.Bq, wl.Bk, windows)
        assert np.array_equal(rp_d.cpu().numpy(), rp) and np.array_equal(ci_d.cpu().numpy(), ci)
        Hm = len(windows)
    else:
        rp, ci = csr
        Hm = wl.H
    out = run_fused(salad, wl, q, k, v, rp, ci, Hm, lam, s).cpu()
    assert torch.isfinite(out.float()).all()
    sel = None if full else stratified_rows(wl, rp, Hm, dense_heads)
    ref = orc.salad_fused(f32(q), f32(k), f32(v), wl.Bq, wl.Bk, rp, ci, Hm, lam, s, sel=sel)
    got = f32(out).reshape(-1, wl.d)
    if sel is not None:
        got = got[sel]
    max_abs, rel = assert_close(got, ref, wl.name, tight=True)
    print(f"\n[parity] {wl.name}: {'whole output' if full else f'{len(sel)} stratified rows'}, "
          f"{got.shape[0]} rows x {wl.d}: max_abs {max_abs:.3e} rel_l2 {rel:.3e}")
    return max_abs, rel


def test_fused_wan13b_90(salad):
    fused_check(salad, wlmod.C2, full=True)                  # every row of every head


def test_fused_wan13b_irregular(salad):
    wl = wlmod.C3
    fused_check(salad, wl, full=True, csr=wlmod.irregular_csr(wl))


def test_fused_wan14b_90(salad):
    fused_check(salad, wlmod.C4)


def test_fused_wan13b_720p_90(salad):
    fused_check(salad, wlmod.C6)


@pytest.mark.parametrize("wl", [wlmod.C5_80, wlmod.C5_90, wlmod.C5_95])
def test_fused_cfg_pair_sparsity_sweep(salad, wl):
    fused_check(salad, wl)


def test_fused_cfg_pair_dense(salad):
    fused_check(salad, wlmod.C5_DENSE, dense_heads=1)        # 512 key blocks per row: the oracle's slowest case


# ------------------------------------------------------------------------------ API behaviour

def test_runs_on_a_side_stream_and_is_deterministic(salad):
    B, H, N, d = 2, 2, 1500, 128
    wl = wlmod.Workload("t", B, H, d, (1, 1, N), 128, 64, (), 1)
    q, k, v = (t.cuda() for t in rand_qkv(B, H, N, d, 77))
    rp, ci = random_csr(wl.nQb, wl.nKb, 5, lo=1, hi=wl.nKb)          # one mask for all heads and batch items
    rp_d, ci_d = dev_csr(rp, ci)
    lam = torch.tensor([0.3, 0.9], dtype=torch.float32, device="cuda")
    s = torch.tensor([0.5, 0.25], dtype=torch.float32, device="cuda")
    ws = salad.alloc_workspace(B, H, N, d)
    side = torch.cuda.Stream()
    outs = []
    for _ in range(2):
        out = torch.empty_like(q)
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            salad.salad_fused_fwd(q, k, v, rp_d, ci_d, 1, lam, s, out=out, workspace=ws, stream=side)
        side.synchronize()
        outs.append(out)
    assert torch.equal(outs[0], outs[1])                               # same launch, same bits
    ref = orc.salad_fused(f32(q.cpu()), f32(k.cpu()), f32(v.cpu()), 128, 64, rp, ci, 1,
                          lam.cpu().numpy(), s.cpu().numpy())
    assert_close(f32(outs[0].cpu()).reshape(-1, d), ref, "side stream")


def test_binding_rejects_bad_tensors(salad):
    q, k, v = (t.cuda() for t in rand_qkv(1, 1, 128, 64, 3))
    rp, ci = dev_csr(*wlmod.dense_csr(1, 2, 1))
    with pytest.raises(ValueError):
        salad.salad_sparse_attn_fwd(q.float(), k, v, rp, ci, 1)                 # not bf16
    with pytest.raises(ValueError):
        salad.salad_sparse_attn_fwd(q, k[:, :, :64], v, rp, ci, 1)               # shape mismatch
    with pytest.raises(salad.SaladError) as err:
        salad.salad_sparse_attn_fwd(q, k, v, rp, ci, 1, Bq=32)                   # unsupported block size
    assert err.value.code in (salad.SALAD_ERR_UNSUPPORTED, salad.SALAD_ERR_WORKSPACE)
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(salad.SaladError) as err:
        salad.salad_sparse_attn_fwd(q, k, v, rp, ci, 1, workspace=small)
    assert err.value.code == salad.SALAD_ERR_WORKSPACE


# ------------------------------------------------------------------------------ scale producer, branch drop

@pytest.mark.parametrize("B,N,D", [(2, 1000, 96), (3, 7, 8), (1, 32760, 1536), (2, 4099, 5120)])
def test_dynamic_scale(salad, B, N, D):
    rng = np.random.default_rng(B * 1000 + D)
    x = bf16(rng.standard_normal((B, N, D)))
    w = (rng.standard_normal(D) * (2.0 / np.sqrt(D))).astype(np.float32)
    got = salad.salad_dynamic_scale(x.cuda(), torch.from_numpy(w).cuda(), bias=-0.2)
    ref = orc.dynamic_scale(f32(x), w, bias=-0.2)
    # fp32 dot products of D terms and a fast exp: a few 1e-6 on a value in (0, 1)
    np.testing.assert_allclose(got.cpu().numpy(), ref, rtol=0, atol=2e-5)
    again = salad.salad_dynamic_scale(x.cuda(), torch.from_numpy(w).cuda(), bias=-0.2)
    assert torch.equal(got, again)                       # fixed reduction order


def test_fused_branch_drop(salad):
    B, H, N, d = 3, 2, 1100, 128
    wl = wlmod.Workload("t", B, H, d, (1, 1, N), 128, 64, (), 1)
    q, k, v = rand_qkv(B, H, N, d, 91)
    rp, ci = random_csr(wl.nQb, wl.nKb, 3, lo=1, hi=wl.nKb)
    rp_d, ci_d = dev_csr(rp, ci)
    lam = np.array([0.7, 0.2], np.float32); s = np.array([0.10, 0.50, 0.90], np.float32)
    lam_d, s_d = torch.from_numpy(lam).cuda(), torch.from_numpy(s).cuda()
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    status = torch.ones(1, dtype=torch.int32, device="cuda")
    drop = salad.salad_fused_fwd(qd, kd, vd, rp_d, ci_d, 1, lam_d, s_d, drop_tau=0.5, status=status)
    status_ok(status)
    ref = orc.salad_fused_drop(f32(q), f32(k), f32(v), 128, 64, rp, ci, 1, lam, s, tau=0.5)
    assert_close(f32(drop.cpu()).reshape(-1, d), ref, "drop")
    sparse = salad.salad_sparse_attn_fwd(qd, kd, vd, rp_d, ci_d, 1)
    full = salad.salad_fused_fwd(qd, kd, vd, rp_d, ci_d, 1, lam_d, s_d)
    assert torch.equal(drop[0], sparse[0])               # below the threshold: the sparse branch, bit for bit
    assert torch.equal(drop[1:], full[1:])               # at or above it: unchanged
    none = salad.salad_fused_fwd(qd, kd, vd, rp_d, ci_d, 1, lam_d, s_d, drop_tau=2.0)
    assert torch.equal(none, sparse)


def test_scale_producer_feeds_the_fused_call(salad):
    # s computed on the device by salad_dynamic_scale goes straight into the attention call
    B, H, N, d, D = 2, 2, 640, 64, 128
    wl = wlmod.Workload("t", B, H, d, (1, 1, N), 64, 64, (), 1)
    q, k, v = rand_qkv(B, H, N, d, 17)
    rng = np.random.default_rng(2)
    x = bf16(rng.standard_normal((B, N, D)))
    w = (rng.standard_normal(D) * 0.3).astype(np.float32)
    rp, ci = random_csr(wl.nQb, wl.nKb, 8, lo=1, hi=wl.nKb)
    rp_d, ci_d = dev_csr(rp, ci)
    lam = np.array([0.4, 0.8], np.float32)
    s_d = salad.salad_dynamic_scale(x.cuda(), torch.from_numpy(w).cuda())
    out = salad.salad_fused_fwd(q.cuda(), k.cuda(), v.cuda(), rp_d, ci_d, 1, torch.from_numpy(lam).cuda(), s_d, Bq=64)
    s_ref = orc.dynamic_scale(f32(x), w)
    ref = orc.salad_fused(f32(q), f32(k), f32(v), 64, 64, rp, ci, 1, lam, s_ref)
    assert_close(f32(out.cpu()).reshape(-1, d), ref, "chain")


# ------------------------------------------------------------------------------ Top-K mask producer

def _check_topk_lists(rp_g, ci_g, rp_o, ci_o, scores, kk):
    """Bit-exact where the selection is unique.  The device scores are fp32, the oracle's fp64: a row
    may differ only where the scores of the swapped blocks agree to fp32 rounding (a near tie), and
    every list must still be a valid selection (kk blocks, ascending, in range)."""
    assert np.array_equal(rp_g, rp_o)
    rows = len(rp_o) - 1
    g = ci_g.reshape(rows, kk); o = ci_o.reshape(rows, kk)
    nKb = scores.shape[-1]
    assert (np.diff(g, axis=1) > 0).all() and g.min() >= 0 and g.max() < nKb
    bad = np.nonzero((g != o).any(axis=1))[0]
    sc = scores.reshape(rows, nKb)
    for r in bad:
        only_g = np.setdiff1d(g[r], o[r]); only_o = np.setdiff1d(o[r], g[r])
        assert len(only_g) == len(only_o)
        tol = 1e-5 * max(1.0, np.abs(sc[r]).max())
        # whatever the device took instead scores within rounding of what the oracle took
        assert np.abs(np.sort(sc[r][only_g]) - np.sort(sc[r][only_o])).max() <= tol, (r, g[r], o[r])
    return len(bad)


@pytest.mark.parametrize("B,H,N,d,Bq,Bk,topk", [
    (1, 2, 1024, 64, 64, 64, 4),
    (2, 3, 1000, 128, 128, 64, 4),      # ragged last blocks on both sides
    (1, 2, 2500, 128, 128, 64, 8),
    (1, 1, 700, 64, 64, 64, 100),       # k above the number of key blocks: dense lists
])
def test_topk_mask_build(salad, B, H, N, d, Bq, Bk, topk):
    q, k, _ = rand_qkv(B, H, N, d, 900 + N)
    rp_o, ci_o, sc = orc.topk_mask(f32(q), f32(k), Bq, Bk, topk, return_scores=True)
    rp_g, ci_g = salad.salad_topk_mask_build(q.cuda(), k.cuda(), topk, Bq=Bq, Bk=Bk)
    kk = min(topk, -(-N // Bk))
    ndiff = _check_topk_lists(rp_g.cpu().numpy(), ci_g.cpu().numpy(), rp_o, ci_o, sc, kk)
    assert ndiff <= max(1, (len(rp_o) - 1) // 50)            # near ties are rare


@pytest.mark.parametrize("N,Bk,topk", [(2048, 64, 5), (6400, 16, 7), (9600, 16, 3), (19200, 16, 9)])      # 32, 400, 600, 1200 key blocks
def test_topk_exact_ties_go_to_the_lower_block(salad, N, Bk, topk):
    # Exact ties: groups of key blocks with identical tokens have bit-identical means and scores, so the
    # selection must be settled by the index (lists equal to the oracle's, no near-tie allowance).  The sizes
    # cover both selection kernels (a row in the registers of one CTA, and the longer rows).
    B, H, d, Bq = 1, 2, 64, 128
    rng = np.random.default_rng(N + topk)
    nKb = N // Bk
    base = rng.standard_normal((B, H, 4, Bk, d)).astype(np.float32)          # four distinct key blocks ...
    which = rng.integers(0, 4, size=nKb)
    k = torch.from_numpy(base[:, :, which].reshape(B, H, N, d)).to(torch.bfloat16)      # ... repeated in random order
    q = torch.from_numpy(rng.standard_normal((B, H, N, d)).astype(np.float32)).to(torch.bfloat16)
    rp_o, ci_o = orc.topk_mask(f32(q), f32(k), Bq, Bk, topk)
    rp_g, ci_g = salad.salad_topk_mask_build(q.cuda(), k.cuda(), topk, Bq=Bq, Bk=Bk)
    assert np.array_equal(rp_g.cpu().numpy(), rp_o)
    assert np.array_equal(ci_g.cpu().numpy(), ci_o)


def test_topk_mask_wan13b_shape(salad):
    # full size, the configuration the benchmark times: k = 51 of 512 key blocks (90 % block sparsity)
    wl = wlmod.C2
    q, k, _ = wlmod.make_qkv(wl)
    rp_o, ci_o, sc = orc.topk_mask(f32(q), f32(k), wl.Bq, wl.Bk, 51, return_scores=True)
    rp_g, ci_g = salad.salad_topk_mask_build(q.cuda(), k.cuda(), 51, Bq=wl.Bq, Bk=wl.Bk)
    ndiff = _check_topk_lists(rp_g.cpu().numpy(), ci_g.cpu().numpy(), rp_o, ci_o, sc, 51)
    assert ndiff <= (len(rp_o) - 1) // 50


def test_topk_mask_feeds_the_fused_call(salad):
    # producer -> consumer on the device with per-(batch, head) lists (Hm = B*H); the oracle runs the
    # same lists the device built, so a near tie cannot fail this test
    B, H, N, d, Bq = 2, 3, 1000, 128, 128
    q, k, v = rand_qkv(B, H, N, d, 77)
    lam = np.array([0.3, 0.8, 0.5], dtype=np.float32); s = np.array([0.6, 0.2], dtype=np.float32)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    rp, ci = salad.salad_topk_mask_build(qd, kd, 5, Bq=Bq)
    status = torch.ones(1, dtype=torch.int32, device="cuda")
    out = salad.salad_fused_fwd(qd, kd, vd, rp, ci, B * H, torch.from_numpy(lam).cuda(), torch.from_numpy(s).cuda(),
                                Bq=Bq, status=status)
    status_ok(status)
    ref = orc.salad_fused(f32(q), f32(k), f32(v), Bq, 64, rp.cpu().numpy(), ci.cpu().numpy(), B * H,
                          lam.astype(np.float64), s.astype(np.float64))
    assert_close(f32(out.cpu()).reshape(-1, d), ref, "fused on top-k lists")
    sp = salad.salad_sparse_attn_fwd(qd, kd, vd, rp, ci, B * H, Bq=Bq)
    ref_s, _ = orc.sparse_attn(f32(q), f32(k), f32(v), Bq, 64, rp.cpu().numpy(), ci.cpu().numpy(), B * H)
    assert_close(f32(sp.cpu()).reshape(-1, d), ref_s, "sparse on top-k lists")


def test_topk_mask_capacity_and_arguments(salad):
    q, k, _ = rand_qkv(1, 1, 256, 64, 3)
    small = torch.empty(3, dtype=torch.int32, device="cuda")
    with pytest.raises(salad.SaladError) as e:
        salad.salad_topk_mask_build(q.cuda(), k.cuda(), 2, Bq=64, col_idx=small)
    assert e.value.code == salad.SALAD_ERR_CAPACITY
    with pytest.raises(salad.SaladError) as e:
        salad.salad_topk_mask_build(q.cuda(), k.cuda(), 0, Bq=64)
    assert e.value.code == salad.SALAD_ERR_INVALID_ARG


# ------------------------------------------------------------------------------ temporal-head permutation

@pytest.mark.parametrize("B,H,grid,d", [(2, 3, (5, 6, 7), 128), (1, 2, (4, 16, 16), 64), (1, 4, (21, 9, 13), 128)])
def test_permute_tokens_bit_exact(salad, B, H, grid, d):
    N = grid[0] * grid[1] * grid[2]
    x, _, _ = rand_qkv(B, H, N, d, 300 + N)
    flags = [(h % 2) == 0 for h in range(H)]
    y = salad.salad_permute_tokens(x.cuda(), grid, flags)
    ref = orc.permute_tokens(f32(x), grid, flags)
    assert np.array_equal(f32(y.cpu()), ref)
    back = salad.salad_permute_tokens(y, grid, flags, inverse=True)
    assert torch.equal(back.cpu(), x)


def test_permuted_sliding_window_pipeline(salad):
    # The paper's ST-SWA: temporal heads are re-ordered, every head then gets a 1-D sliding window,
    # the output goes back to the original order.  Device pipeline against the oracle's.
    grid = (8, 8, 16)                     # N = 1024
    B, H, N, d, Bq = 1, 4, 1024, 128, 128
    q, k, v = rand_qkv(B, H, N, d, 55)
    flags = [1, 0, 1, 0]                  # heads 0 and 2 temporal
    windows = [(0, 0, 64), (0, 0, 200), (0, 0, 24), (0, 0, 130)]       # 1-D half-widths per head
    lam = np.array([0.5, 0.1, 0.9, 0.3], dtype=np.float32); s = np.array([0.4], dtype=np.float32)
    qd, kd, vd = (salad.salad_permute_tokens(t.cuda(), grid, flags) for t in (q, k, v))
    rp, ci = salad.salad_mask_build(1, 1, N, Bq, 64, windows)
    out_p = salad.salad_fused_fwd(qd, kd, vd, rp, ci, H, torch.from_numpy(lam).cuda(), torch.from_numpy(s).cuda(), Bq=Bq)
    out = salad.salad_permute_tokens(out_p, grid, flags, inverse=True)
    qo, ko, vo = (orc.permute_tokens(f32(t), grid, flags) for t in (q, k, v))
    rp_o, ci_o = orc.mask_build(1, 1, N, Bq, 64, windows)
    assert np.array_equal(rp.cpu().numpy(), rp_o) and np.array_equal(ci.cpu().numpy(), ci_o)
    ref_p = orc.salad_fused(qo, ko, vo, Bq, 64, rp_o, ci_o, H, lam.astype(np.float64), s.astype(np.float64))
    ref = orc.permute_tokens(ref_p.reshape(B, H, N, d), grid, flags, inverse=True)
    assert_close(f32(out.cpu()).reshape(-1, d), ref.reshape(-1, d), "permuted ST-SWA")


def _stswa_oracle(q, k, v, grid, flags, windows, lam, s, kq, ks):
    """The oracle's ST-SWA pipeline: re-order the temporal heads, a 1-D window on every head's own order (blocks of
    128 x 64 tokens, or of the tokens of kq x ks whole spatial positions), Algorithm 1, order restored."""
    T = grid[0]
    B, H, N, d = q.shape
    qp, kp, vp = (orc.permute_tokens(f32(t), grid, flags) for t in (q, k, v))
    ref_p = np.empty((B, H, N, d))
    lists = {}
    for h in range(H):
        Bq, Bk = (kq * T, ks * T) if flags[h] else (128, 64)
        rp, ci = orc.mask_build(1, 1, N, Bq, Bk, [(0, 0, windows[h])])
        lists[h] = (rp, ci)
        r = orc.salad_fused(qp[:, h:h + 1], kp[:, h:h + 1], vp[:, h:h + 1], Bq, Bk, rp, ci, 1,
                            lam[h:h + 1].astype(np.float64), s.astype(np.float64))
        ref_p[:, h] = r.reshape(B, N, d)
    return orc.permute_tokens(ref_p, grid, flags, inverse=True), lists


@pytest.mark.parametrize("grid,B,H,d,flags,windows", [
    ((21, 6, 10), 1, 4, 128, [1, 0, 1, 0], [100, 200, 300, 90]),       # T = 21: blocks of 3 and 6 positions (63, 126 tokens)
    ((8, 8, 16), 2, 3, 64, [0, 1, 1], [64, 130, 40]),                  # T = 8: 8 and 16 positions fill the tiles exactly
    ((5, 7, 9), 1, 2, 128, [1, 1], [33, 400]),                         # 63 positions: ragged last blocks on both sides
])
def test_stswa_through_the_loads(salad, grid, B, H, d, flags, windows):
    # The paper's ST-SWA with the re-ordering done by the loads and stores of the attention kernel: lists
    # bit-exact against the oracle's 1-D window masks, output against the oracle's permute / attend / permute-back.
    T, Hs, Ws = grid
    N = T * Hs * Ws
    q, k, v = rand_qkv(B, H, N, d, 1200 + N)
    rng = np.random.default_rng(N)
    lam = rng.uniform(0.2, 1, H).astype(np.float32); s = rng.uniform(0.2, 0.9, B).astype(np.float32)
    rows, kq, ks, nkb_p = salad.salad_stswa_blocks(grid)
    assert (kq, ks) == (128 // T, 64 // T)
    rp_d, ci_d = salad.salad_stswa_mask_build(grid, flags, windows)
    ref, lists = _stswa_oracle(q, k, v, grid, flags, windows, lam, s, kq, ks)
    rp_g, ci_g = rp_d.cpu().numpy(), ci_d.cpu().numpy()
    for h in range(H):
        rp_o, ci_o = lists[h]
        n_own = len(rp_o) - 1
        got_rp = rp_g[h * rows:h * rows + n_own + 1] - rp_g[h * rows]
        assert np.array_equal(got_rp, rp_o), h
        assert np.array_equal(ci_g[rp_g[h * rows]:rp_g[h * rows + n_own]], ci_o), h
        assert (np.diff(rp_g[h * rows + n_own:(h + 1) * rows + 1]) == 0).all()       # rows beyond the head's blocks: empty
    status = torch.ones(1, dtype=torch.int32, device="cuda")
    out = torch.full_like(q.cuda(), 3.0)
    salad.salad_fused_stswa_fwd(q.cuda(), k.cuda(), v.cuda(), grid, flags, rp_d, ci_d, torch.from_numpy(lam).cuda(),
                                torch.from_numpy(s).cuda(), out=out, status=status)
    status_ok(status)
    assert_close(f32(out.cpu()).reshape(-1, d), ref.reshape(-1, d), "ST-SWA through the loads")


def test_stswa_wan13b_shape(salad):
    # ST-SWA through the loads at the full Wan-1.3B shape, as the benchmark runs it (every second head temporal,
    # a window of a tenth of the sequence on every head's own order): lists bit-exact for every head, output on
    # sampled rows of every head -- first, last and random query blocks, first / last / random row of each.
    wl = wlmod.C2
    grid = wl.grid
    T, Hs, Ws = grid
    B, H, N, d = wl.B, wl.H, wl.N, wl.d
    flags = [h % 2 for h in range(H)]
    windows = [N // 20] * H
    q, k, v = wlmod.make_qkv(wl)
    lam, s = wlmod.make_scales(wl)
    rows, kq, ks, nkb_p = salad.salad_stswa_blocks(grid)
    rp_d, ci_d = salad.salad_stswa_mask_build(grid, flags, windows)
    rp_g, ci_g = rp_d.cpu().numpy(), ci_d.cpu().numpy()
    status = torch.ones(1, dtype=torch.int32, device="cuda")
    out = torch.full_like(q.cuda(), 3.0)
    salad.salad_fused_stswa_fwd(q.cuda(), k.cuda(), v.cuda(), grid, flags, rp_d, ci_d, torch.from_numpy(lam).cuda(),
                                torch.from_numpy(s).cuda(), out=out, status=status)
    status_ok(status)
    got_all = f32(out.cpu())
    assert np.isfinite(got_all).all()
    # position m of a temporal head's own order holds token order_t[m] (from the oracle's re-ordering of an index ramp)
    ramp = np.arange(N, dtype=np.float32).reshape(1, 1, N, 1)
    order_t = orc.permute_tokens(ramp, grid, [1]).reshape(N).astype(np.int64)
    qp, kp, vp = (orc.permute_tokens(f32(t), grid, flags) for t in (q, k, v))
    rng = np.random.default_rng(77)
    worst = (0.0, 0.0)
    for h in range(H):
        Bq, Bk = (kq * T, ks * T) if flags[h] else (128, 64)
        rp_o, ci_o = orc.mask_build(1, 1, N, Bq, Bk, [(0, 0, windows[h])])
        n_own = len(rp_o) - 1
        assert np.array_equal(rp_g[h * rows:h * rows + n_own + 1] - rp_g[h * rows], rp_o), h
        assert np.array_equal(ci_g[rp_g[h * rows]:rp_g[h * rows + n_own]], ci_o), h
        blocks = {0, n_own - 1} | set(rng.integers(0, n_own, 6).tolist())
        ms = []
        for i in blocks:
            m0, m1 = i * Bq, min(N, (i + 1) * Bq)
            ms += [m0, m1 - 1, int(rng.integers(m0, m1))]
        ms = np.unique(np.asarray(ms, dtype=np.int64))
        ref = orc.salad_fused(qp[:, h:h + 1], kp[:, h:h + 1], vp[:, h:h + 1], Bq, Bk, rp_o, ci_o, 1,
                              lam[h:h + 1].astype(np.float64), s.astype(np.float64), sel=ms)     # B = 1: row index = m
        toks = order_t[ms] if flags[h] else ms
        ma, rel = assert_close(got_all[0, h, toks], ref, f"ST-SWA full size, head {h}", tight=True)
        worst = (max(worst[0], ma), max(worst[1], rel))
    print(f"\n[parity] ST-SWA through the loads, {wl.name}: max_abs {worst[0]:.3e} rel_l2 {worst[1]:.3e}")


# ------------------------------------------------------------------------------ full projection (Alg. 1 level 1)

@pytest.mark.parametrize("B,H,N,d,with_bias", [
    (1, 2, 300, 128, True),        # one output tile, ragged token tile
    (2, 3, 1000, 128, False),      # D = 384: the second column tile is half empty
    (1, 12, 520, 64, True),        # D = 768, four heads per column tile
    (1, 12, 2048, 128, True),      # the 1.3B width, several tiles per SM none
])
def test_proj_combine(salad, B, H, N, d, with_bias):
    rng = np.random.default_rng(500 + N)
    D = H * d
    o_s = bf16(rng.standard_normal((B, H, N, d))); o_l = bf16(rng.standard_normal((B, H, N, d)))
    w = bf16(rng.standard_normal((D, D)) / np.sqrt(D))
    bias = torch.from_numpy(rng.standard_normal(D).astype(np.float32)) if with_bias else None
    s = torch.from_numpy(rng.uniform(0.2, 0.9, B).astype(np.float32))
    status = torch.ones(1, dtype=torch.int32, device="cuda")
    out = salad.salad_proj_combine_fwd(o_s.cuda(), o_l.cuda(), w.cuda(), s.cuda(),
                                       bias.cuda() if with_bias else None, status=status)
    status_ok(status)
    ref = orc.proj_combine(f32(o_s), f32(o_l), f32(w), s.numpy().astype(np.float64),
                           bias.numpy() if with_bias else None)
    assert_close(f32(out.cpu()).reshape(-1, d), ref.reshape(-1, d), "proj_combine")
    # in place on O_s, and the zero-initialised layer returns the sparse branch bit for bit
    buf = o_s.cuda().clone()
    salad.salad_proj_combine_fwd(buf, o_l.cuda(), w.cuda(), s.cuda(), bias.cuda() if with_bias else None, out=buf)
    assert torch.equal(buf, out)
    zero = salad.salad_proj_combine_fwd(o_s.cuda(), o_l.cuda(), torch.zeros_like(w).cuda(), s.cuda())
    assert torch.equal(zero.cpu(), o_s)


def test_full_projection_pipeline_matches_fused_for_block_diagonal(salad):
    # sparse call + linear call + projection with W = blockdiag(lambda_h I) against the one-pass fused call
    wl = wlmod.C1
    q, k, v = wlmod.make_qkv(wl)
    T, Hs, Ws = wl.grid
    lam, s = wlmod.make_scales(wl)
    rp, ci = salad.salad_mask_build(T, Hs, Ws, wl.Bq, wl.Bk, wl.windows)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    lam_d, s_d = torch.from_numpy(lam).cuda(), torch.from_numpy(s).cuda()
    fused = salad.salad_fused_fwd(qd, kd, vd, rp, ci, len(wl.windows), lam_d, s_d, Bq=wl.Bq, Bk=wl.Bk)
    o_s = salad.salad_sparse_attn_fwd(qd, kd, vd, rp, ci, len(wl.windows), Bq=wl.Bq, Bk=wl.Bk)
    o_l = salad.salad_linear_attn_fwd(qd, kd, vd)
    w = torch.from_numpy(np.kron(np.diag(lam.astype(np.float64)), np.eye(wl.d))).to(torch.bfloat16).cuda()
    out = salad.salad_proj_combine_fwd(o_s, o_l, w, s_d)
    # lambda rounded to bf16 in W and O_l rounded to bf16 between the calls: not bit-equal, but close
    assert_close(f32(out.cpu()).reshape(-1, wl.d), f32(fused.cpu()).reshape(-1, wl.d).astype(np.float64), "pipeline vs fused")


@pytest.mark.parametrize("B,H,N,d,Bq", [(2, 3, 1000, 128, 128), (1, 2, 1024, 64, 64), (1, 12, 700, 128, 128)])
def test_fused_block_projection(salad, B, H, N, d, Bq):
    # one d x d projection block per head folded into the linear state (Alg. 1 Level 1 without head mixing)
    wl = wlmod.Workload("t", B, H, d, (1, 1, N), Bq, 64, (), 1)
    q, k, v = rand_qkv(B, H, N, d, 600 + N)
    rng = np.random.default_rng(N + d)
    rp, ci = random_csr(wl.nQb, wl.nKb, 4 + N, lo=0, hi=min(wl.nKb, 9))
    rp_d, ci_d = dev_csr(rp, ci)
    wb = bf16(rng.standard_normal((H, d, d)) / np.sqrt(d))
    s = rng.uniform(0.2, 0.9, B).astype(np.float32)
    qd, kd, vd, s_d = q.cuda(), k.cuda(), v.cuda(), torch.from_numpy(s).cuda()
    status = torch.ones(1, dtype=torch.int32, device="cuda")
    out = salad.salad_fused_proj_fwd(qd, kd, vd, rp_d, ci_d, 1, wb.cuda(), s_d, Bq=Bq, status=status)
    status_ok(status)
    ref = orc.salad_fused_blockproj(f32(q), f32(k), f32(v), Bq, 64, rp, ci, 1, f32(wb), s.astype(np.float64))
    assert_close(f32(out.cpu()).reshape(-1, d), ref, "block projection")
    # W_h = lambda_h I is the per-head scalar of salad_fused_fwd (lambda representable in bf16: same bits up to
    # the order of the roundings), zero blocks are the sparse branch bit for bit
    lam = torch.tensor([0.5, 0.25, 1.0, 0.75] * 3)[:H]
    wi = torch.stack([l * torch.eye(d) for l in lam]).to(torch.bfloat16).cuda()
    a = salad.salad_fused_proj_fwd(qd, kd, vd, rp_d, ci_d, 1, wi, s_d, Bq=Bq)
    b_ = salad.salad_fused_fwd(qd, kd, vd, rp_d, ci_d, 1, lam.float().cuda(), s_d, Bq=Bq)
    assert_close(f32(a.cpu()).reshape(-1, d), f32(b_.cpu()).reshape(-1, d).astype(np.float64), "identity blocks vs scalar")
    zero = salad.salad_fused_proj_fwd(qd, kd, vd, rp_d, ci_d, 1, torch.zeros_like(wi), s_d, Bq=Bq)
    sparse = salad.salad_sparse_attn_fwd(qd, kd, vd, rp_d, ci_d, 1, Bq=Bq)
    assert torch.equal(zero, sparse)
    # the drop threshold
    drop = salad.salad_fused_proj_fwd(qd, kd, vd, rp_d, ci_d, 1, wb.cuda(), s_d, Bq=Bq, drop_tau=2.0)
    assert torch.equal(drop, sparse)


def test_fused_block_projection_wan13b_shape(salad):
    # the block projection at the full Wan-1.3B shape (the benchmark's configuration), stratified rows of all heads
    wl = wlmod.C2
    q, k, v = wlmod.make_qkv(wl)
    T, Hs, Ws = wl.grid
    _, s = wlmod.make_scales(wl)
    rng = np.random.default_rng(4242)
    wb = bf16(rng.standard_normal((wl.H, wl.d, wl.d)) / np.sqrt(wl.d))
    rp_d, ci_d = salad.salad_mask_build(T, Hs, Ws, wl.Bq, wl.Bk, wl.windows)
    rp, ci = rp_d.cpu().numpy(), ci_d.cpu().numpy()
    Hm = len(wl.windows)
    status = torch.ones(1, dtype=torch.int32, device="cuda")
    out = salad.salad_fused_proj_fwd(q.cuda(), k.cuda(), v.cuda(), rp_d, ci_d, Hm, wb.cuda(), torch.from_numpy(s).cuda(),
                                     Bq=wl.Bq, Bk=wl.Bk, status=status)
    status_ok(status)
    sel = stratified_rows(wl, rp, Hm, dense_heads=2)
    ref = orc.salad_fused_blockproj(f32(q), f32(k), f32(v), wl.Bq, wl.Bk, rp, ci, Hm, f32(wb), s.astype(np.float64), sel=sel)
    max_abs, rel = assert_close(f32(out.cpu()).reshape(-1, wl.d)[sel], ref, "block projection, full size", tight=True)
    print(f"\n[parity] block projection, {wl.name}: {len(sel)} stratified rows: max_abs {max_abs:.3e} rel_l2 {rel:.3e}")


def test_state_pass_as_its_own_call_on_a_side_stream(salad):
    # the reductions of Eq. 3 on one stream, the attention call on another, ordered by an event: the same bits
    # as the one-call path, and the state against the oracle
    B, H, N, d = 2, 3, 3000, 128
    q, k, v = rand_qkv(B, H, N, d, 41)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    rp, ci = random_csr(-(-N // 128), -(-N // 64), 6, lo=1, hi=12)
    rp_d, ci_d = dev_csr(rp, ci)
    lam = torch.rand(H, device="cuda"); s = torch.tensor([0.3, 0.8], device="cuda")
    whole = salad.salad_fused_fwd(qd, kd, vd, rp_d, ci_d, 1, lam, s, drop_tau=0.5)
    ws = salad.alloc_workspace(B, H, N, d)
    kv = torch.empty((B, H, d, d), dtype=torch.float32, device="cuda"); z = torch.empty((B, H, d), dtype=torch.float32, device="cuda")
    st1 = torch.ones(1, dtype=torch.int32, device="cuda"); st2 = torch.ones(1, dtype=torch.int32, device="cuda")
    side, main = torch.cuda.Stream(), torch.cuda.current_stream()
    side.wait_stream(main)
    salad.salad_linear_state_fwd(kd, vd, ws, kv_out=kv, z_out=z, status=st1, stream=side)
    done = torch.cuda.Event(); done.record(side)
    main.wait_event(done)
    out = salad.salad_fused_prepared_fwd(qd, kd, vd, rp_d, ci_d, 1, lam, s, ws, status=st2, drop_tau=0.5)
    torch.cuda.synchronize()
    assert int(st1.item()) == 0 and int(st2.item()) == 0
    assert torch.equal(out, whole)
    kv_ref, z_ref = orc.linear_state(f32(k), f32(v))
    np.testing.assert_allclose(z.cpu().numpy(), z_ref, rtol=1e-4, atol=1e-3)
    np.testing.assert_allclose(kv.cpu().numpy(), kv_ref, rtol=1e-3, atol=np.abs(kv_ref).max() * 1e-4)


# ------------------------------------------------------------------------------ degenerate sizes

@pytest.mark.parametrize("B,H,N,d,Bq", [
    (1, 1, 1, 64, 64),          # a single token
    (1, 2, 63, 128, 128),       # less than one key block
    (3, 1, 65, 64, 128),        # one token into the second key block
    (5, 1, 129, 128, 64),       # one row into the third query block, odd number of query blocks
    (1, 20, 200, 64, 64),       # many heads, short sequence
    (4, 48, 330, 64, 128),      # more (batch, head) pairs than SMs: one state chunk per head, 192 state CTAs
    (2, 80, 700, 128, 128),     # 160 heads at d = 128: the state kernel runs in more than one wave
])
def test_fused_degenerate_sizes(salad, B, H, N, d, Bq):
    q, k, v = rand_qkv(B, H, N, d, 700 + N)
    nQb, nKb = -(-N // Bq), -(-N // 64)
    rp, ci = random_csr(nQb, nKb, 3 + N, lo=0, hi=nKb)
    rp_d, ci_d = dev_csr(rp, ci)
    lam = np.linspace(0.2, 0.9, H).astype(np.float32); s = np.linspace(0.3, 0.7, B).astype(np.float32)
    status = torch.ones(1, dtype=torch.int32, device="cuda")
    out = salad.salad_fused_fwd(q.cuda(), k.cuda(), v.cuda(), rp_d, ci_d, 1, torch.from_numpy(lam).cuda(),
                                torch.from_numpy(s).cuda(), Bq=Bq, status=status)
    status_ok(status)
    ref = orc.salad_fused(f32(q), f32(k), f32(v), Bq, 64, rp, ci, 1, lam.astype(np.float64), s.astype(np.float64))
    assert_close(f32(out.cpu()).reshape(-1, d), ref, "degenerate fused")
    lin = salad.salad_linear_attn_fwd(q.cuda(), k.cuda(), v.cuda())
    assert_close(f32(lin.cpu()).reshape(-1, d), orc.linear_attn(f32(q), f32(k), f32(v)), "degenerate linear")


def test_fused_with_no_kept_block_at_all_is_the_scaled_linear_branch(salad):
    B, H, N, d = 1, 2, 640, 128
    q, k, v = rand_qkv(B, H, N, d, 12)
    nQb = -(-N // 128)
    rp = np.zeros(nQb + 1, dtype=np.int32); ci = np.zeros(0, dtype=np.int32)
    rp_d, ci_d = dev_csr(rp, ci)
    lam = np.array([0.5, 0.25], dtype=np.float32); s = np.array([0.5], dtype=np.float32)
    out = salad.salad_fused_fwd(q.cuda(), k.cuda(), v.cuda(), rp_d, ci_d, 1, torch.from_numpy(lam).cuda(),
                                torch.from_numpy(s).cuda())
    ref = orc.linear_attn(f32(q), f32(k), f32(v)).reshape(B, H, N, d) * (lam * s[0])[None, :, None, None]
    assert_close(f32(out.cpu()).reshape(-1, d), ref.reshape(-1, d), "linear only through the fused call")


def test_long_sequence_linear_and_sparse_band(salad):
    # 256k tokens of one head: the longest sequence the tests run; a narrow band keeps the oracle cheap
    B, H, N, d = 1, 1, 262144, 128
    rng = np.random.default_rng(99)
    q, k, v = (bf16(rng.standard_normal((B, H, N, d))) for _ in range(3))
    rp_d, ci_d = salad.salad_mask_build(1, 1, N, 128, 64, [(0, 0, 100)])
    lam = torch.tensor([0.5], device="cuda"); s = torch.tensor([0.5], device="cuda")
    status = torch.ones(1, dtype=torch.int32, device="cuda")
    out = salad.salad_fused_fwd(q.cuda(), k.cuda(), v.cuda(), rp_d, ci_d, 1, lam, s, status=status)
    status_ok(status)
    wl = wlmod.Workload("long", B, H, d, (1, 1, N), 128, 64, ((0, 0, 100),), 0)
    sel = np.concatenate([np.arange(0, 130), np.arange(N - 130, N), wlmod.sample_rows(wl, 300)])
    ref = orc.salad_fused(f32(q), f32(k), f32(v), 128, 64, rp_d.cpu().numpy(), ci_d.cpu().numpy(), 1,
                          np.array([0.5]), np.array([0.5]), sel=sel)
    got = f32(out.cpu()).reshape(-1, d)[sel]
    assert_close(got, ref, "long sequence")


# ------------------------------------------------------------------------------ bounded waits

def test_an_expired_wait_is_reported_and_the_context_stays_usable(salad):
    # Nothing faults here: a one-thread kernel waits 2 ms on a barrier nobody arrives on, gives up and
    # writes the time-out code, the way every wait inside the compute kernels does.
    status, waited = salad.salad_selftest_bounded_wait()
    torch.cuda.synchronize()
    assert int(status.item()) == salad.SALAD_ERR_TIMEOUT
    assert 2_000_000 <= int(waited.item()) < 50_000_000
    # the context is fine: a compute call right after it runs and matches the oracle
    wl = wlmod.C1
    q, k, v = wlmod.make_qkv(wl)
    out = salad.salad_linear_attn_fwd(q.cuda(), k.cuda(), v.cuda())
    assert_close(f32(out.cpu()).reshape(-1, wl.d), orc.linear_attn(f32(q), f32(k), f32(v)), "after time-out")


# ------------------------------------------------------------------------------ seeded random sweeps

def test_mask_random_grids_bit_exact(salad):
    rng = np.random.default_rng(2024)
    for _ in range(25):
        T, Hs, Ws = int(rng.integers(1, 7)), int(rng.integers(1, 10)), int(rng.integers(1, 12))
        Bq = int(rng.choice([4, 8, 16, 32, 64, 128])); Bk = int(rng.choice([4, 8, 16, 32, 64]))
        Hm = int(rng.integers(1, 4))
        windows = [(int(rng.integers(0, T + 1)), int(rng.integers(0, Hs + 1)), int(rng.integers(0, Ws + 1)))
                   for _ in range(Hm)]
        rp, ci = salad.salad_mask_build(T, Hs, Ws, Bq, Bk, windows)
        rp_ref, ci_ref = orc.mask_build(T, Hs, Ws, Bq, Bk, windows)
        assert np.array_equal(rp.cpu().numpy(), rp_ref), (T, Hs, Ws, Bq, Bk, windows)
        assert np.array_equal(ci.cpu().numpy()[:len(ci_ref)], ci_ref), (T, Hs, Ws, Bq, Bk, windows)


def test_fused_random_shapes(salad):
    rng = np.random.default_rng(4048)
    for case in range(10):
        B, H = int(rng.integers(1, 3)), int(rng.integers(1, 4))
        N = int(rng.integers(1, 1400)); d = int(rng.choice([64, 128])); Bq = int(rng.choice([64, 128]))
        Hm = int(rng.choice([1, H, B * H]))
        q, k, v = rand_qkv(B, H, N, d, 9000 + case)
        nQb, nKb = -(-N // Bq), -(-N // 64)
        rp, ci = random_csr(Hm * nQb, nKb, 77 + case, lo=0, hi=nKb)
        rp_d, ci_d = dev_csr(rp, ci)
        lam = rng.uniform(0, 1, H).astype(np.float32); s = rng.uniform(0, 1, B).astype(np.float32)
        status = torch.ones(1, dtype=torch.int32, device="cuda")
        out = salad.salad_fused_fwd(q.cuda(), k.cuda(), v.cuda(), rp_d, ci_d, Hm, torch.from_numpy(lam).cuda(),
                                    torch.from_numpy(s).cuda(), Bq=Bq, status=status)
        status_ok(status)
        ref = orc.salad_fused(f32(q), f32(k), f32(v), Bq, 64, rp, ci, Hm, lam.astype(np.float64), s.astype(np.float64))
        assert_close(f32(out.cpu()).reshape(-1, d), ref, f"random case {case}: B{B} H{H} N{N} d{d} Bq{Bq} Hm{Hm}")


def test_two_streams_with_their_own_workspaces(salad):
    # calls that may overlap on the GPU need separate workspaces and status words; results must not change
    B, H, N, d = 1, 4, 2048, 128
    q, k, v = (t.cuda() for t in rand_qkv(B, H, N, d, 808))
    rp, ci = salad.salad_mask_build(4, 16, 32, 128, 64, [(1, 3, 8)])
    lam = torch.rand(H, device="cuda"); s = torch.rand(B, device="cuda")
    serial_f = salad.salad_fused_fwd(q, k, v, rp, ci, 1, lam, s)
    serial_l = salad.salad_linear_attn_fwd(q, k, v)
    torch.cuda.synchronize()
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    ws_a = salad.alloc_workspace(B, H, N, d); ws_b = salad.alloc_workspace(B, H, N, d)
    st_a = torch.ones(1, dtype=torch.int32, device="cuda"); st_b = torch.ones(1, dtype=torch.int32, device="cuda")
    out_a = torch.empty_like(q); out_b = torch.empty_like(q)
    for _ in range(10):
        salad.salad_fused_fwd(q, k, v, rp, ci, 1, lam, s, out=out_a, workspace=ws_a, status=st_a, stream=sa)
        salad.salad_linear_attn_fwd(q, k, v, out=out_b, workspace=ws_b, status=st_b, stream=sb)
    torch.cuda.synchronize()
    assert int(st_a.item()) == 0 and int(st_b.item()) == 0
    assert torch.equal(out_a, serial_f) and torch.equal(out_b, serial_l)


def test_fused_call_in_a_cuda_graph(salad):
    # the call allocates nothing and synchronises nothing: it can be captured and replayed
    B, H, N, d = 1, 4, 2048, 128
    q, k, v = (t.cuda() for t in rand_qkv(B, H, N, d, 909))
    rp, ci = salad.salad_mask_build(4, 16, 32, 128, 64, [(1, 3, 8)])
    lam = torch.rand(H, device="cuda"); s = torch.rand(B, device="cuda")
    ws = salad.alloc_workspace(B, H, N, d)
    status = torch.ones(1, dtype=torch.int32, device="cuda")
    eager = salad.salad_fused_fwd(q, k, v, rp, ci, 1, lam, s, workspace=ws, status=status)      # also the first-call set-up
    torch.cuda.synchronize()
    out = torch.zeros_like(q)
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            salad.salad_fused_fwd(q, k, v, rp, ci, 1, lam, s, out=out, workspace=ws, status=status, stream=side)
    for _ in range(3):
        out.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert torch.equal(out, eager)


def test_calls_do_not_depend_on_the_workspace_contents(salad):
    # the first kernel of every call clears the status words; nothing else is read before it is written
    B, H, N, d = 1, 3, 1500, 128
    q, k, v = (t.cuda() for t in rand_qkv(B, H, N, d, 321))
    rp, ci = random_csr(-(-N // 128), -(-N // 64), 5, lo=1, hi=8)
    rp_d, ci_d = dev_csr(rp, ci)
    lam = torch.rand(H, device="cuda"); s = torch.rand(B, device="cuda")
    clean = salad.alloc_workspace(B, H, N, d); clean.zero_()
    # every word of the dirty workspace is -1: the status words read "failed", the launch-order region holds
    # out-of-range block ids, the states and partials NaN patterns.  (The fused call reads the order list
    # without a dependency wait of its own, relying on the ordering of the launches before it: a stale list
    # would show here as a difference.)
    dirty = torch.full_like(clean, 0xFF)
    for fn in (lambda ws, st: salad.salad_linear_attn_fwd(q, k, v, workspace=ws, status=st),
               lambda ws, st: salad.salad_fused_fwd(q, k, v, rp_d, ci_d, 1, lam, s, workspace=ws, status=st),
               lambda ws, st: salad.salad_sparse_attn_fwd(q, k, v, rp_d, ci_d, 1, workspace=ws, status=st)):
        st_a = torch.full((1,), 77, dtype=torch.int32, device="cuda"); st_b = st_a.clone()
        a = fn(clean, st_a); b = fn(dirty, st_b)
        torch.cuda.synchronize()
        assert int(st_a.item()) == 0 and int(st_b.item()) == 0
        assert torch.equal(a, b)



# ------------------------------------------------------------------------------ mask validation

def _valid_lists(rows, nKb, seed):
    rp, ci = random_csr(rows, nKb, seed, lo=1, hi=min(nKb, 6))
    return rp, ci


def test_csr_validator_accepts_valid_lists_and_rejects_each_kind_of_corruption(salad):
    rows, nKb = 40, 24
    rp, ci = _valid_lists(rows, nKb, 1)
    ok = salad.salad_csr_validate(*dev_csr(rp, ci), nKb)
    torch.cuda.synchronize()
    assert int(ok.item()) == 0
    # builder output and all-kept lists are valid too
    brp, bci = salad.salad_mask_build(4, 16, 16, 64, 64, [(1, 1, 1), (0, 5, 5)])
    assert int(salad.salad_csr_validate(brp, bci, 16).item()) == 0
    empty_rows = np.zeros(rows + 1, np.int32)
    assert int(salad.salad_csr_validate(*dev_csr(empty_rows, np.zeros(0, np.int32)), nKb).item()) == 0

    def corrupt(fn):
        r2, c2 = rp.copy(), ci.copy()
        fn(r2, c2)
        st = salad.salad_csr_validate(*dev_csr(r2, c2), nKb)
        torch.cuda.synchronize()
        return int(st.item())

    mid = rows // 2
    def first_offset(r, c): r[0] = 1
    def decreasing(r, c): r[mid] = r[mid - 1] - 1
    def past_capacity(r, c): r[rows] = len(c) + 5
    def huge_offset(r, c): r[mid:] = 2**31 - 1                    # must not be followed into col_idx
    def negative_offset(r, c): r[3] = -4
    def col_too_large(r, c): c[r[mid]] = nKb
    def col_negative(r, c): c[r[mid]] = -1
    def duplicate(r, c):
        i = next(i for i in range(rows) if r[i + 1] - r[i] >= 2); c[r[i] + 1] = c[r[i]]
    def unsorted_(r, c):
        i = next(i for i in range(rows) if r[i + 1] - r[i] >= 2); c[r[i]], c[r[i] + 1] = c[r[i] + 1], c[r[i]]
    for fn in (first_offset, decreasing, past_capacity, huge_offset, negative_offset, col_too_large, col_negative,
               duplicate, unsorted_):
        assert corrupt(fn) == salad.SALAD_ERR_BAD_MASK, fn.__name__


def test_attention_calls_reject_a_broken_mask_without_touching_the_output(salad):
    # Offsets that decrease are caught by the first kernel of every call with a sparse branch; the full check
    # (here: block ids out of order) runs when the caller has switched it on.  In both cases the attention
    # kernels do nothing: the prefilled output stays as it was.  Nothing here reads out of bounds: the broken
    # lists stay inside their arrays.
    B, H, N, d = 1, 2, 1024, 128
    q, k, v = (t.cuda() for t in rand_qkv(B, H, N, d, 5))
    nQb, nKb = N // 128, N // 64
    rp, ci = random_csr(nQb, nKb, 9, lo=2, hi=6)
    lam = torch.rand(H, device="cuda"); s = torch.rand(B, device="cuda")
    good = salad.salad_fused_fwd(q, k, v, *dev_csr(rp, ci), 1, lam, s)
    bad_rp = rp.copy(); bad_rp[3], bad_rp[4] = rp[4], rp[3]                 # decreasing offsets
    for call in ("sparse", "fused"):
        out = torch.full_like(q, 7.0)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        if call == "sparse":
            salad.salad_sparse_attn_fwd(q, k, v, *dev_csr(bad_rp, ci), 1, out=out, status=status)
        else:
            salad.salad_fused_fwd(q, k, v, *dev_csr(bad_rp, ci), 1, lam, s, out=out, status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == salad.SALAD_ERR_BAD_MASK
        assert (out == 7.0).all()
    # opt-in full validation: swapped block ids inside a row
    bad_ci = ci.copy(); bad_ci[rp[2]], bad_ci[rp[2] + 1] = ci[rp[2] + 1], ci[rp[2]]
    out = torch.full_like(q, 7.0)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    salad.salad_set_mask_validation(len(ci))
    try:
        salad.salad_fused_fwd(q, k, v, *dev_csr(rp, bad_ci), 1, lam, s, out=out, status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == salad.SALAD_ERR_BAD_MASK and (out == 7.0).all()
        # valid lists pass through the same path and give the same bits as without the check
        again = salad.salad_fused_fwd(q, k, v, *dev_csr(rp, ci), 1, lam, s, status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0 and torch.equal(again, good)
    finally:
        salad.salad_set_mask_validation(0)
    # and the context is fine afterwards
    after = salad.salad_fused_fwd(q, k, v, *dev_csr(rp, ci), 1, lam, s, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and torch.equal(after, good)
