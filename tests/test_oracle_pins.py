"""Pins of the CPU oracle against things other than itself: the equations written out as
dense N x N matrices in numpy, torch's SDPA routine, closed forms and hand-counted masks.
CPU only."""
import os

import numpy as np
import pytest
import torch

from oracle import salad_oracle as orc
from paper_2601_16515_b200 import workloads as wlmod


def bf16_round(a):
    return torch.from_numpy(np.asarray(a, dtype=np.float32)).to(torch.bfloat16).float().numpy()


def rand_qkv(B, H, N, d, seed, scale=1.0):
    rng = np.random.default_rng(seed)
    return tuple(bf16_round(rng.standard_normal((B, H, N, d)) * scale) for _ in range(3))


def token_mask_from_csr(N, Bq, Bk, row_ptr, col_idx, hm, nQb):
    """Matrix M of Eq. 2 as a boolean 'allowed' matrix [N, N]."""
    allowed = np.zeros((N, N), dtype=bool)
    for i in range(nQb):
        r = hm * nQb + i
        for j in col_idx[row_ptr[r]:row_ptr[r + 1]]:
            allowed[i * Bq:min(N, (i + 1) * Bq), j * Bk:min(N, (j + 1) * Bk)] = True
    return allowed


def dense_masked_softmax(q, k, v, allowed):
    """Eq. 2 literally: softmax((Q K^T + M)/sqrt(d)) V with M in {-inf, 0}."""
    d = q.shape[-1]
    M = np.where(allowed, 0.0, -np.inf)
    s = (q.astype(np.float64) @ k.astype(np.float64).T + M) / np.sqrt(d)
    s = s - s.max(axis=1, keepdims=True)
    p = np.exp(s)
    p /= p.sum(axis=1, keepdims=True)
    return p @ v.astype(np.float64)


# ----------------------------------------------------------------------------- mask

def window_mask_vectorised(T, Hs, Ws, Bq, Bk, win):
    """Token-level window mask by broadcasting, then 'any' over blocks."""
    N = T * Hs * Ws
    n = np.arange(N)
    t, h, w = n // (Hs * Ws), (n // Ws) % Hs, n % Ws
    tok = ((np.abs(t[:, None] - t[None, :]) <= win[0]) &
           (np.abs(h[:, None] - h[None, :]) <= win[1]) &
           (np.abs(w[:, None] - w[None, :]) <= win[2]))
    nQb, nKb = -(-N // Bq), -(-N // Bk)
    blk = np.zeros((nQb, nKb), dtype=bool)
    for i in range(nQb):
        for j in range(nKb):
            blk[i, j] = tok[i * Bq:(i + 1) * Bq, j * Bk:(j + 1) * Bk].any()
    return blk


def csr_to_dense(row_ptr, col_idx, rows, nKb):
    out = np.zeros((rows, nKb), dtype=bool)
    for r in range(rows):
        out[r, col_idx[row_ptr[r]:row_ptr[r + 1]]] = True
    return out


def test_mask_hand_counted():
    # Grid 2 x 2 x 4, blocks of 4 tokens = one (t,h) row each; block id = 2 t + h.
    rp, ci = orc.mask_build(2, 2, 4, 4, 4, [(0, 0, 1)])      # same row only
    assert rp.tolist() == [0, 1, 2, 3, 4] and ci.tolist() == [0, 1, 2, 3]
    rp, ci = orc.mask_build(2, 2, 4, 4, 4, [(0, 1, 0)])      # both rows of the own frame
    assert rp.tolist() == [0, 2, 4, 6, 8] and ci.tolist() == [0, 1, 0, 1, 2, 3, 2, 3]
    rp, ci = orc.mask_build(2, 2, 4, 4, 4, [(1, 0, 0)])      # same row in both frames
    assert ci.tolist() == [0, 2, 1, 3, 0, 2, 1, 3]
    # Bq = 8 (one frame per query block), Bk = 4, two mask heads
    rp, ci = orc.mask_build(2, 2, 4, 8, 4, [(0, 0, 0), (1, 0, 0)])
    assert rp.tolist() == [0, 2, 4, 8, 12]
    assert ci.tolist() == [0, 1, 2, 3, 0, 1, 2, 3, 0, 1, 2, 3]


@pytest.mark.parametrize("grid,Bq,Bk,win", [
    ((3, 5, 7), 16, 8, (1, 1, 2)),     # ragged: N = 105
    ((4, 6, 6), 32, 16, (0, 2, 2)),
    ((4, 6, 6), 16, 16, (2, 0, 0)),
    ((2, 9, 11), 64, 32, (1, 3, 4)),   # N = 198
])
def test_mask_vs_vectorised_token_mask(grid, Bq, Bk, win):
    T, Hs, Ws = grid
    rp, ci = orc.mask_build(T, Hs, Ws, Bq, Bk, [win])
    ref = window_mask_vectorised(T, Hs, Ws, Bq, Bk, win)
    got = csr_to_dense(rp, ci, ref.shape[0], ref.shape[1])
    assert (got == ref).all()
    for r in range(ref.shape[0]):                             # ascending, unique
        row = ci[rp[r]:rp[r + 1]]
        assert (np.diff(row) > 0).all()


def test_mask_invariants_tiny_config():
    wl = wlmod.C1
    T, Hs, Ws = wl.grid
    rp, ci = orc.mask_build(T, Hs, Ws, wl.Bq, wl.Bk, wl.windows)
    nQb, nKb = wl.nQb, wl.nKb
    dense = csr_to_dense(rp, ci, 2 * nQb, nKb)
    assert dense.sum() == 2 * nQb * 4                         # exactly 25 % kept per row
    for i in range(nQb):
        frame = i // 4
        assert dense[i].nonzero()[0].tolist() == [4 * frame + c for c in range(4)]
        assert dense[nQb + i].nonzero()[0].tolist() == [4 * f + i % 4 for f in range(4)]
    # window >= grid keeps everything; window 0 keeps exactly the overlapping key blocks
    rp, ci = orc.mask_build(T, Hs, Ws, 128, 64, [(T, Hs, Ws)])
    assert len(ci) == (wl.N // 128) * (wl.N // 64)
    rp, ci = orc.mask_build(T, Hs, Ws, 128, 64, [(0, 0, 0)])
    assert ci.tolist() == list(range(wl.N // 64))


def test_mask_block_counts_wan_shape():
    # Block counts for the 21 x 30 x 52 grid with 128 x 64 blocks; sparsity targets of the
    # workload list: ~80 %, ~90 %, ~95 %.
    total = 256 * 512
    for win, lo, hi in [((5, 5, 24), 0.79, 0.81), ((2, 5, 24), 0.895, 0.905), ((1, 4, 24), 0.94, 0.955)]:
        rp, ci = orc.mask_build(21, 30, 52, 128, 64, [win])
        sp = 1.0 - len(ci) / total
        assert lo <= sp <= hi, (win, sp)
        # own blocks always kept
        for i in (0, 100, 255):
            row = ci[rp[i]:rp[i + 1]]
            assert 2 * i in row and min(2 * i + 1, 511) in row


# ----------------------------------------------------------------------------- sparse branch

@pytest.mark.parametrize("N,Bq,Bk,d", [(256, 64, 64, 64), (200, 64, 32, 32), (300, 128, 64, 128)])
def test_sparse_vs_dense_masked_softmax(N, Bq, Bk, d):
    B, H = 1, 2
    q, k, v = rand_qkv(B, H, N, d, 11)
    nQb, nKb = -(-N // Bq), -(-N // Bk)
    rng = np.random.default_rng(5)
    rp, cols = [0], []
    for r in range(H * nQb):
        row = np.sort(rng.choice(nKb, size=rng.integers(1, nKb + 1), replace=False))
        cols.append(row); rp.append(rp[-1] + len(row))
    rp = np.asarray(rp, np.int32); ci = np.concatenate(cols).astype(np.int32)
    o, lse = orc.sparse_attn(q, k, v, Bq, Bk, rp, ci, H)
    o = o.reshape(B, H, N, d)
    for h in range(H):
        allowed = token_mask_from_csr(N, Bq, Bk, rp, ci, h, nQb)
        ref = dense_masked_softmax(q[0, h], k[0, h], v[0, h], allowed)
        np.testing.assert_allclose(o[0, h], ref, rtol=1e-10, atol=1e-12)
        # library routine as a second witness
        sd = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(q[0, h]).double()[None], torch.from_numpy(k[0, h]).double()[None],
            torch.from_numpy(v[0, h]).double()[None], attn_mask=torch.from_numpy(allowed)[None])
        np.testing.assert_allclose(o[0, h], sd[0].numpy(), rtol=1e-9, atol=1e-11)
        # lse: log of the masked row sums of exp(scores)
        s = (q[0, h].astype(np.float64) @ k[0, h].astype(np.float64).T) / np.sqrt(d)
        ref_lse = np.log(np.where(allowed, np.exp(s), 0.0).sum(axis=1))
        np.testing.assert_allclose(lse.reshape(B, H, N)[0, h], ref_lse, rtol=1e-10)


def test_sparse_all_kept_is_full_attention():
    B, H, N, d = 2, 2, 192, 64
    q, k, v = rand_qkv(B, H, N, d, 3)
    rp, ci = wlmod.dense_csr(-(-N // 64), -(-N // 64), 1)
    o, _ = orc.sparse_attn(q, k, v, 64, 64, rp, ci, 1)
    o = o.reshape(B, H, N, d)
    s = np.einsum("bhnd,bhmd->bhnm", q.astype(np.float64), k.astype(np.float64)) / np.sqrt(d)
    p = np.exp(s - s.max(-1, keepdims=True)); p /= p.sum(-1, keepdims=True)
    ref = np.einsum("bhnm,bhmd->bhnd", p, v.astype(np.float64))            # Eq. 1
    np.testing.assert_allclose(o, ref, rtol=1e-10, atol=1e-12)


def test_sparse_closed_forms():
    B, H, N, d, Bq, Bk = 1, 1, 200, 32, 64, 32
    q, k, v = rand_qkv(B, H, N, d, 9)
    T = 1
    rp, ci = orc.mask_build(1, 1, N, Bq, Bk, [(0, 0, 40)])
    nQb = -(-N // Bq)
    # K = 0: uniform weights -> O_s is the mean of V over the kept tokens, lse = log(count)
    o, lse = orc.sparse_attn(q, np.zeros_like(k), v, Bq, Bk, rp, ci, 1)
    allowed = token_mask_from_csr(N, Bq, Bk, rp, ci, 0, nQb)
    cnt = allowed.sum(1)
    ref = (allowed[:, :, None] * v[0, 0][None].astype(np.float64)).sum(1) / cnt[:, None]
    np.testing.assert_allclose(o, ref, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(lse, np.log(cnt), rtol=1e-12)
    # V = const: the output is that constant whatever the weights are
    vc = np.broadcast_to(bf16_round(np.linspace(-1, 1, d)), v.shape).copy()
    o, _ = orc.sparse_attn(q, k, vc, Bq, Bk, rp, ci, 1)
    np.testing.assert_allclose(o, np.broadcast_to(vc[0, 0, 0], o.shape), rtol=1e-12, atol=1e-13)
    # one key with a dominant score: O_s of every row that sees it -> that key's V row
    kd = k.copy(); qd = np.abs(q)
    kd[0, 0, 70] = 64.0
    o, _ = orc.sparse_attn(qd, kd, v, Bq, Bk, rp, ci, 1)
    sees = allowed[:, 70]
    np.testing.assert_allclose(o[sees], np.broadcast_to(v[0, 0, 70], o[sees].shape), atol=1e-6)
    # empty rows: zero output, lse = -inf
    rp0 = np.zeros(nQb + 1, np.int32)
    o, lse = orc.sparse_attn(q, k, v, Bq, Bk, rp0, np.zeros(0, np.int32), 1)
    assert (o == 0).all() and np.isneginf(lse).all()


def test_sparse_row_selection_matches_full():
    B, H, N, d = 2, 3, 130, 32
    q, k, v = rand_qkv(B, H, N, d, 4)
    rp, ci = orc.mask_build(1, 10, 13, 32, 16, [(0, 2, 3)] * H)
    full, lse_full = orc.sparse_attn(q, k, v, 32, 16, rp, ci, H)
    sel = np.array([0, 5, 129, 130, 777, B * H * N - 1], dtype=np.int64)
    part, lse = orc.sparse_attn(q, k, v, 32, 16, rp, ci, H, sel=sel)
    np.testing.assert_array_equal(part, full[sel])
    np.testing.assert_array_equal(lse, lse_full[sel])


# ----------------------------------------------------------------------------- linear branch

def test_linear_vs_explicit_quadratic_form():
    B, H, N, d = 2, 2, 150, 32
    q, k, v = rand_qkv(B, H, N, d, 21)
    o = orc.linear_attn(q, k, v, eps=0.0).reshape(B, H, N, d)
    fq, fk = np.maximum(q, 0).astype(np.float64), np.maximum(k, 0).astype(np.float64)
    W = np.einsum("bhnd,bhmd->bhnm", fq, fk)                    # phi(Q) phi(K)^T, N x N
    ref = (W @ v.astype(np.float64)) / W.sum(-1, keepdims=True)
    np.testing.assert_allclose(o, ref, rtol=1e-10, atol=1e-12)
    kv, z = orc.linear_state(k, v)
    np.testing.assert_allclose(kv, np.einsum("bhna,bhnc->bhac", fk, v.astype(np.float64)), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(z, fk.sum(2), rtol=1e-12)
    # KV is not symmetric in (key channel, value channel): guard against a transposed state
    assert not np.allclose(kv, np.swapaxes(kv, -1, -2))


def test_linear_closed_forms():
    B, H, N, d = 1, 2, 97, 16
    q, k, v = rand_qkv(B, H, N, d, 22)
    # V = const c -> O_l = c wherever the denominator is positive
    vc = np.broadcast_to(bf16_round(np.linspace(-2, 2, d)), v.shape).copy()
    o = orc.linear_attn(q, k, vc, eps=0.0)
    np.testing.assert_allclose(o, np.broadcast_to(vc[0, 0, 0], o.shape), rtol=1e-12, atol=1e-13)
    # K = const >= 0 -> uniform weights -> O_l = mean of V
    kc = np.full_like(k, 0.5)
    o = orc.linear_attn(q, kc, v, eps=0.0).reshape(B, H, N, d)
    ref = np.broadcast_to(v.astype(np.float64).mean(2, keepdims=True), o.shape)
    np.testing.assert_allclose(o, ref, rtol=1e-11, atol=1e-13)
    # Q <= 0 everywhere -> numerator and denominator vanish -> 0 (eps defines 0/0)
    o = orc.linear_attn(-np.abs(q), k, v, eps=1e-6)
    assert (o == 0).all()
    # ... and without eps the quotient 0/0 is taken as 0 as well, never NaN; rows with a positive
    # denominator are untouched by that rule
    qz = q.copy(); qz[:, :, ::3] = -np.abs(qz[:, :, ::3])
    o0 = orc.linear_attn(qz, k, v, eps=0.0).reshape(B, H, N, d)
    assert np.isfinite(o0).all() and (o0[:, :, ::3] == 0).all()
    np.testing.assert_array_equal(o0[:, :, 1::3], orc.linear_attn(q, k, v, eps=0.0).reshape(B, H, N, d)[:, :, 1::3])
    # homogeneity: phi(a K) = a phi(K) for a > 0 cancels between numerator and denominator
    o1 = orc.linear_attn(q, k, v, eps=0.0)
    o2 = orc.linear_attn(q, 4.0 * k, v, eps=0.0)
    np.testing.assert_allclose(o1, o2, rtol=1e-12, atol=1e-13)
    # eps enters only the denominator
    kv, z = orc.linear_state(k, v)
    fq = np.maximum(q, 0).astype(np.float64)
    num = np.einsum("bhna,bhac->bhnc", fq, kv); den = np.einsum("bhna,bha->bhn", fq, z)
    o3 = orc.linear_attn(q, k, v, eps=0.25).reshape(B, H, N, d)
    np.testing.assert_allclose(o3, num / (den[..., None] + 0.25), rtol=1e-12, atol=1e-13)


# ----------------------------------------------------------------------------- combination

def test_fused_is_sparse_plus_scaled_linear():
    wl = wlmod.C1
    q, k, v = (t.float().numpy() for t in wlmod.make_qkv(wl))
    T, Hs, Ws = wl.grid
    rp, ci = orc.mask_build(T, Hs, Ws, wl.Bq, wl.Bk, wl.windows)
    lam, s = wlmod.make_scales(wl)
    o_s, _ = orc.sparse_attn(q, k, v, wl.Bq, wl.Bk, rp, ci, wl.Hm)
    o_l = orc.linear_attn(q, k, v)
    fused = orc.salad_fused(q, k, v, wl.Bq, wl.Bk, rp, ci, wl.Hm, lam, s)
    c = np.repeat((s.astype(np.float64)[:, None] * lam.astype(np.float64)[None, :]).reshape(-1), wl.N)[:, None]
    np.testing.assert_allclose(fused, o_s + c * o_l, rtol=1e-13, atol=1e-14)
    # zero scale (zero-initialised projection / dropped branch) -> exactly the sparse branch
    z = orc.salad_fused(q, k, v, wl.Bq, wl.Bk, rp, ci, wl.Hm, np.zeros_like(lam), s)
    np.testing.assert_array_equal(z, o_s)
    # lambda = s = 1 -> plain sum; and the result is linear in the scale
    one = orc.salad_fused(q, k, v, wl.Bq, wl.Bk, rp, ci, wl.Hm, np.ones_like(lam), np.ones_like(s))
    np.testing.assert_allclose(one, o_s + o_l, rtol=1e-13, atol=1e-14)
    half = orc.salad_fused(q, k, v, wl.Bq, wl.Bk, rp, ci, wl.Hm, 0.5 * np.ones_like(lam), np.ones_like(s))
    np.testing.assert_allclose(half - o_s, 0.5 * (one - o_s), rtol=1e-9, atol=1e-12)
    # per-head / per-batch indexing of the scales (B = 2, distinct values)
    B, H, N, d = 2, 3, 64, 16
    q2, k2, v2 = rand_qkv(B, H, N, d, 8)
    rp2, ci2 = wlmod.dense_csr(1, 1, 1)
    lam2 = np.array([0.1, 0.5, 0.9]); s2 = np.array([0.25, 0.75])
    f2 = orc.salad_fused(q2, k2, v2, 64, 64, rp2, ci2, 1, lam2, s2).reshape(B, H, N, d)
    os2 = orc.sparse_attn(q2, k2, v2, 64, 64, rp2, ci2, 1)[0].reshape(B, H, N, d)
    ol2 = orc.linear_attn(q2, k2, v2).reshape(B, H, N, d)
    for b in range(B):
        for h in range(H):
            np.testing.assert_allclose(f2[b, h], os2[b, h] + s2[b] * lam2[h] * ol2[b, h], rtol=1e-13, atol=1e-14)


# ----------------------------------------------------------------------------- input generators

def test_workloads_are_seeded_and_sliceable():
    wl = wlmod.C1
    a = wlmod.make_qkv(wl); b = wlmod.make_qkv(wl)
    for x, y in zip(a, b):
        assert torch.equal(x, y)
    sub = wlmod.make_qkv(wl, heads=[1])
    assert torch.equal(sub[0][:, 0], a[0][:, 1])
    small = wlmod.Workload("s", 1, 2, 32, (3, 10, 12), 128, 64, (), 7, irregular=True)
    rp, ci = wlmod.irregular_csr(small, 0.3, 0.6)
    assert rp[-1] == len(ci) and len(rp) == small.H * small.nQb + 1
    for r in range(len(rp) - 1):
        row = ci[rp[r]:rp[r + 1]]
        assert (np.diff(row) > 0).all() and row.min() >= 0 and row.max() < small.nKb
        i = r % small.nQb
        assert 2 * i in row


# ----------------------------------------------------------------------------- scale producer, branch drop

def test_dynamic_scale_pins():
    rng = np.random.default_rng(31)
    B, N, D = 3, 257, 96
    x = bf16_round(rng.standard_normal((B, N, D)))
    w = bf16_round(rng.standard_normal(D) * 0.2)
    s = orc.dynamic_scale(x, w, bias=0.3)
    z = np.einsum("bnd,d->bn", x.astype(np.float64), w.astype(np.float64)) + 0.3
    ref = torch.sigmoid(torch.from_numpy(z)).mean(dim=1).numpy()          # library sigmoid as witness
    np.testing.assert_allclose(s, ref, rtol=1e-12)
    assert ((s > 0) & (s < 1)).all()                                       # the paper's s in (0, 1)
    # closed forms: w = 0 -> sigmoid(bias); x -> -x with zero bias -> 1 - s
    np.testing.assert_allclose(orc.dynamic_scale(x, np.zeros(D), bias=0.0), 0.5, rtol=1e-15)
    np.testing.assert_allclose(orc.dynamic_scale(x, np.zeros(D), bias=2.0), 1 / (1 + np.exp(-2.0)), rtol=1e-14)
    np.testing.assert_allclose(orc.dynamic_scale(-x, w) + orc.dynamic_scale(x, w), 1.0, rtol=1e-13)
    # a mean over tokens, per batch item: permuting tokens changes nothing, batch items are independent
    perm = rng.permutation(N)
    np.testing.assert_allclose(orc.dynamic_scale(x[:, perm], w), orc.dynamic_scale(x, w), rtol=1e-13)
    np.testing.assert_allclose(orc.dynamic_scale(x[1:2], w, 0.3), s[1:2], rtol=1e-15)


def test_fused_branch_drop_pins():
    B, H, N, d = 3, 2, 128, 32
    q, k, v = rand_qkv(B, H, N, d, 41)
    rp, ci = wlmod.dense_csr(2, 2, 1)
    lam = np.array([0.7, 0.2]); s = np.array([0.10, 0.50, 0.90])
    full = orc.salad_fused(q, k, v, 64, 64, rp, ci, 1, lam, s).reshape(B, H, N, d)
    sparse = orc.sparse_attn(q, k, v, 64, 64, rp, ci, 1)[0].reshape(B, H, N, d)
    drop = orc.salad_fused_drop(q, k, v, 64, 64, rp, ci, 1, lam, s, tau=0.5).reshape(B, H, N, d)
    np.testing.assert_array_equal(drop[0], sparse[0])          # s < tau: exactly the sparse branch
    np.testing.assert_array_equal(drop[1], full[1])            # s == tau is kept ("below" is dropped)
    np.testing.assert_array_equal(drop[2], full[2])
    np.testing.assert_array_equal(orc.salad_fused_drop(q, k, v, 64, 64, rp, ci, 1, lam, s, tau=-1.0).reshape(B, H, N, d), full)
    np.testing.assert_array_equal(orc.salad_fused_drop(q, k, v, 64, 64, rp, ci, 1, lam, s, tau=2.0).reshape(B, H, N, d), sparse)


# ----------------------------------------------------------------------------- Top-K block mask

def _golden(name):
    out = {}
    for line in open(os.path.join(os.path.dirname(__file__), "golden", name)):
        if line.startswith("#") or not line.strip():
            continue
        key, *vals = line.split()
        out[key] = np.array([float(v) for v in vals])
    return out


def test_topk_mask_hand_example():
    g = _golden("topk_hand_example.txt")
    q = g["Q"].reshape(1, 1, 6, 1)
    for kname in ("K", "K2"):
        k = g[kname].reshape(1, 1, 6, 1)
        rp, ci, sc = orc.topk_mask(q, k, 2, 2, 2, return_scores=True)
        assert rp.tolist() == [0, 2, 4, 6]
        assert ci.tolist() == g["TOP2_" + kname].astype(int).tolist()
        assert orc.topk_mask(q, k, 2, 2, 1)[1].tolist() == g["TOP1_" + kname].astype(int).tolist()
        if kname == "K":
            np.testing.assert_allclose(sc.reshape(-1), g["SCORES_K"], rtol=0, atol=1e-15)


def test_topk_mask_matches_per_token_brute_force():
    # Step 2 taken literally: every query token's similarity with the key-block means, averaged
    # over the tokens of the query block, then argsort.  Ragged last blocks on both sides.
    rng = np.random.default_rng(77)
    B, H, N, d, Bq, Bk, topk = 2, 3, 150, 16, 32, 16, 3
    q = bf16_round(rng.standard_normal((B, H, N, d))); k = bf16_round(rng.standard_normal((B, H, N, d)))
    rp, ci, sc = orc.topk_mask(q, k, Bq, Bk, topk, return_scores=True)
    nQb, nKb = -(-N // Bq), -(-N // Bk)
    assert len(rp) == B * H * nQb + 1 and (np.diff(rp) == topk).all()
    q64, k64 = q.astype(np.float64), k.astype(np.float64)
    for b in range(B):
        for h in range(H):
            kbar = np.stack([k64[b, h, j * Bk:(j + 1) * Bk].mean(0) for j in range(nKb)])       # [nKb, d]
            tok = q64[b, h] @ kbar.T                                                          # [N, nKb]
            for i in range(nQb):
                s = tok[i * Bq:(i + 1) * Bq].mean(0)
                np.testing.assert_allclose(sc[b * H + h, i], s, rtol=1e-12, atol=1e-13)
                want = np.sort(np.argsort(-s, kind="stable")[:topk])
                r = (b * H + h) * nQb + i
                assert ci[rp[r]:rp[r + 1]].tolist() == want.tolist()


def test_topk_mask_special_cases():
    rng = np.random.default_rng(78)
    B, H, N, d, Bq, Bk = 1, 2, 128, 8, 32, 16
    q = bf16_round(rng.standard_normal((B, H, N, d))); k = bf16_round(rng.standard_normal((B, H, N, d)))
    nQb, nKb = N // Bq, N // Bk
    # k >= number of key blocks: everything is kept, i.e. the dense lists
    rp, ci = orc.topk_mask(q, k, Bq, Bk, nKb + 5)
    drp, dci = wlmod.dense_csr(nQb, nKb, B * H)
    assert rp.tolist() == drp.tolist() and ci.tolist() == dci.tolist()
    # a planted key block: its tokens all equal c * qbar_i, c large -> query block i must select it
    k2 = k.copy()
    i, j = 2, 5
    qbar = q[0, 1, i * Bq:(i + 1) * Bq].astype(np.float64).mean(0)
    k2[0, 1, j * Bk:(j + 1) * Bk] = bf16_round(50.0 * qbar)
    rp2, ci2 = orc.topk_mask(q, k2, Bq, Bk, 1)
    assert ci2[(1 * nQb + i)] == j
    # positive rescaling of the queries changes no selection; heads and batch items are independent
    rp3, ci3 = orc.topk_mask(4.0 * q, k, Bq, Bk, 3)
    assert ci3.tolist() == orc.topk_mask(q, k, Bq, Bk, 3)[1].tolist()
    sub = orc.topk_mask(q[:, 1:2], k[:, 1:2], Bq, Bk, 3)[1]
    assert sub.tolist() == orc.topk_mask(q, k, Bq, Bk, 3)[1].reshape(H, -1)[1].tolist()


def test_sparse_attn_with_per_batch_and_head_masks():
    # Hm = B*H: head (b, h) uses list block b*H + h.  Against a dense masked softmax built per head.
    rng = np.random.default_rng(79)
    B, H, N, d, Bq, Bk = 2, 2, 64, 8, 16, 16
    q, k, v = rand_qkv(B, H, N, d, 79)
    rp, ci = orc.topk_mask(q, k, Bq, Bk, 2)
    out = orc.sparse_attn(q, k, v, Bq, Bk, rp, ci, B * H)[0].reshape(B, H, N, d)
    nQb = N // Bq
    for b in range(B):
        for h in range(H):
            M = np.full((N, N), -np.inf)
            for i in range(nQb):
                r = (b * H + h) * nQb + i
                for j in ci[rp[r]:rp[r + 1]]:
                    M[i * Bq:(i + 1) * Bq, j * Bk:(j + 1) * Bk] = 0.0
            x = q[b, h].astype(np.float64) @ k[b, h].astype(np.float64).T / np.sqrt(d) + M
            p = np.exp(x - x.max(1, keepdims=True)); p /= p.sum(1, keepdims=True)
            np.testing.assert_allclose(out[b, h], p @ v[b, h].astype(np.float64), rtol=1e-10, atol=1e-12)


# ----------------------------------------------------------------------------- temporal-head permutation

def test_temporal_order_hand_example_and_inverse():
    # T = 2 frames of a 1 x 3 grid: tokens (t, s) = 0:(0,0) 1:(0,1) 2:(0,2) 3:(1,0) 4:(1,1) 5:(1,2);
    # grouped by spatial location: (0,0) (1,0) (0,1) (1,1) (0,2) (1,2) = tokens 0 3 1 4 2 5
    assert orc.temporal_order((2, 1, 3)).tolist() == [0, 3, 1, 4, 2, 5]
    rng = np.random.default_rng(5)
    grid = (3, 2, 4)
    x = rng.standard_normal((2, 3, 24, 4)).astype(np.float32)
    flags = [1, 0, 1]
    y = orc.permute_tokens(x, grid, flags)
    assert np.array_equal(y[:, 1], x[:, 1])                                  # unflagged head untouched
    assert not np.array_equal(y[:, 0], x[:, 0])
    assert np.array_equal(orc.permute_tokens(y, grid, flags, inverse=True), x)
    # temporal neighbours become adjacent: positions m, m+1 (same s) are one frame apart
    perm = orc.temporal_order(grid)
    S = grid[1] * grid[2]
    d = np.diff(perm.reshape(S, grid[0]), axis=1)
    assert (d == S).all()


def test_attention_commutes_with_the_permutation():
    # attention is equivariant under a joint re-ordering of the tokens of Q, K, V: dense attention
    # on the permuted tensors, un-permuted, equals dense attention on the originals
    grid = (4, 2, 4)
    B, H, N, d = 1, 2, 32, 8
    q, k, v = rand_qkv(B, H, N, d, 91)
    flags = [1, 1]
    qp, kp, vp = (orc.permute_tokens(t, grid, flags) for t in (q, k, v))
    rp, ci = wlmod.dense_csr(2, 2, 1)
    o_perm = orc.sparse_attn(qp, kp, vp, 16, 16, rp, ci, 1)[0].reshape(B, H, N, d)
    o_ref = orc.sparse_attn(q, k, v, 16, 16, rp, ci, 1)[0].reshape(B, H, N, d)
    np.testing.assert_allclose(orc.permute_tokens(o_perm, grid, flags, inverse=True), o_ref, rtol=1e-12, atol=1e-14)
    # and the 1-D window on the permuted order reaches temporal neighbours the same window misses on
    # the original order: token (t, s) and (t+1, s) are 1 apart after, Hs*Ws apart before
    perm = orc.temporal_order(grid)
    pos = np.empty_like(perm); pos[perm] = np.arange(len(perm))
    assert abs(pos[0 * 8 + 3] - pos[1 * 8 + 3]) == 1


# ----------------------------------------------------------------------------- full projection (Alg. 1 level 1)

def test_proj_combine_pins():
    rng = np.random.default_rng(101)
    B, H, N, d = 2, 3, 37, 8
    D = H * d
    o_s = rng.standard_normal((B, H, N, d)).astype(np.float32)
    o_l = rng.standard_normal((B, H, N, d)).astype(np.float32)
    w = (rng.standard_normal((D, D)) * 0.2).astype(np.float32)
    bias = rng.standard_normal(D).astype(np.float32)
    s = np.array([0.3, 0.8])
    got = orc.proj_combine(o_s, o_l, w, s, bias)
    # the definition with library routines: concatenate heads, y = x W^T + b, split heads again
    x = np.transpose(o_l.astype(np.float64), (0, 2, 1, 3)).reshape(B, N, D)
    y = x @ w.astype(np.float64).T + bias.astype(np.float64)
    y = np.transpose(y.reshape(B, N, H, d), (0, 2, 1, 3))
    np.testing.assert_allclose(got, o_s + s[:, None, None, None] * y, rtol=1e-12, atol=1e-13)
    # zero-initialised layer: the sparse branch exactly (the starting point of tuning, Sec. 4.2)
    assert np.array_equal(orc.proj_combine(o_s, o_l, np.zeros((D, D), np.float32), s), o_s.astype(np.float64))
    # identity: the plain residual sum
    np.testing.assert_allclose(orc.proj_combine(o_s, o_l, np.eye(D, dtype=np.float32), s),
                               o_s + s[:, None, None, None] * o_l.astype(np.float64), rtol=1e-14)
    # a matrix that moves head 1 to head 0 and nothing else
    w2 = np.zeros((D, D), np.float32); w2[0:d, d:2 * d] = np.eye(d)
    out2 = orc.proj_combine(o_s, o_l, w2, np.ones(B))
    np.testing.assert_allclose(out2[:, 0], o_s[:, 0].astype(np.float64) + o_l[:, 1], rtol=1e-14)
    assert np.array_equal(out2[:, 1:], o_s[:, 1:].astype(np.float64))


def test_proj_combine_block_diagonal_is_the_fused_path():
    # Proj = blockdiag(lambda_h I_d) turns the full projection into the per-head static scale of the
    # fused call: O_s + s_b * lambda_h * O_l
    B, H, N, d = 2, 2, 64, 16
    q, k, v = rand_qkv(B, H, N, d, 103)
    rp, ci = wlmod.dense_csr(4, 4, 1)
    lam = np.array([0.7, 0.2]); s = np.array([0.4, 0.9])
    o_s = orc.sparse_attn(q, k, v, 16, 16, rp, ci, 1)[0].reshape(B, H, N, d)
    o_l = orc.linear_attn(q, k, v).reshape(B, H, N, d)
    w = np.kron(np.diag(lam), np.eye(d))
    got = orc.proj_combine(o_s, o_l, w, s)
    # o_s and o_l pass through fp32 in the wrapper: compare at that precision
    ref = orc.salad_fused(q, k, v, 16, 16, rp, ci, 1, lam, s).reshape(B, H, N, d)
    np.testing.assert_allclose(got, ref, rtol=1e-6, atol=1e-6)


def test_stswa_with_blocks_of_whole_spatial_positions():
    # The reading behind salad_fused_stswa_fwd for heads with temporal locality (Appendix A.1): tokens grouped by
    # spatial position, m = s*T + t; a key block = the T tokens of ks positions, a query block those of kq
    # positions; a block pair is kept iff some token pair is within w of each other in the re-ordered sequence.
    # The oracle's composition (permute, 1-D window mask with blocks of kq*T x ks*T tokens, Eq. 2, permute back)
    # against the same thing written from first principles on (t, s) coordinates with a dense N x N mask.
    T, Hs, Ws, kq, ks, w, d = 3, 2, 5, 2, 1, 4, 8
    S, N = Hs * Ws, T * Hs * Ws
    grid = (T, Hs, Ws)
    q, k, v = rand_qkv(1, 1, N, d, 301)
    qp, kp, vp = (orc.permute_tokens(t, grid, [1]) for t in (q, k, v))
    rp, ci = orc.mask_build(1, 1, N, kq * T, ks * T, [(0, 0, w)])
    o_p, _ = orc.sparse_attn(qp, kp, vp, kq * T, ks * T, rp, ci, 1)
    got = orc.permute_tokens(o_p.reshape(1, 1, N, d), grid, [1], inverse=True)[0, 0]
    # first principles: positions in the re-ordered sequence, block ids from spatial positions
    n = np.arange(N); t, sp = n // S, n % S
    m = sp * T + t
    qblk, kblk = sp // kq, sp // ks
    nQb, nKb = -(-S // kq), -(-S // ks)
    kept = np.zeros((nQb, nKb), bool)
    for a in range(N):
        for b_ in range(N):
            if abs(int(m[a]) - int(m[b_])) <= w:
                kept[qblk[a], kblk[b_]] = True
    allow = kept[qblk][:, kblk]                                 # [N, N] over original token ids
    sc = (q[0, 0].astype(np.float64) @ k[0, 0].astype(np.float64).T) / np.sqrt(d)
    sc = np.where(allow, sc, -np.inf)
    p = np.exp(sc - sc.max(1, keepdims=True)); p /= p.sum(1, keepdims=True)
    np.testing.assert_allclose(got, p @ v[0, 0].astype(np.float64), rtol=1e-10, atol=1e-12)
    assert 0 < allow.mean() < 1                                 # a real mask, not all-kept


def test_blockproj_pins():
    # One d x d projection block per head (Alg. 1 Level 1 without head mixing), pinned from both sides:
    # against the full projection with a block-diagonal weight, and against the per-head scalar.
    B, H, N, d = 2, 3, 48, 8
    q, k, v = rand_qkv(B, H, N, d, 105)
    rng = np.random.default_rng(7)
    rp, ci = wlmod.dense_csr(3, 6, 1)                     # 16 x 8 blocks, everything kept
    s = np.array([0.4, 0.9])
    wb = (rng.standard_normal((H, d, d)) * 0.4).astype(np.float32)
    assert not np.allclose(wb, np.swapaxes(wb, 1, 2))     # a transposed block must not pass
    got = orc.salad_fused_blockproj(q, k, v, 16, 8, rp, ci, 1, wb, s).reshape(B, H, N, d)
    o_s = orc.sparse_attn(q, k, v, 16, 8, rp, ci, 1)[0].reshape(B, H, N, d)
    o_l = orc.linear_attn(q, k, v).reshape(B, H, N, d)
    # ... written out with numpy: y[c] = sum_a W_h[c][a] x[a]
    want = o_s + s[:, None, None, None] * np.einsum("hca,bhna->bhnc", wb.astype(np.float64), o_l)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-13)
    # ... the full projection layer whose weight is zero outside the diagonal blocks (o_s, o_l pass through
    # fp32 in that wrapper: compared at that precision)
    W = np.zeros((H * d, H * d), np.float32)
    for h in range(H):
        W[h * d:(h + 1) * d, h * d:(h + 1) * d] = wb[h]
    np.testing.assert_allclose(got, orc.proj_combine(o_s, o_l, W, s), rtol=1e-5, atol=1e-6)
    # ... W_h = lambda_h I: the per-head static scale of the fused call
    lam = np.array([0.7, 0.2, 1.3])
    wl_ = np.stack([l * np.eye(d) for l in lam]).astype(np.float32)
    np.testing.assert_allclose(orc.salad_fused_blockproj(q, k, v, 16, 8, rp, ci, 1, wl_, s),
                               orc.salad_fused(q, k, v, 16, 8, rp, ci, 1, lam.astype(np.float32), s), rtol=1e-6, atol=1e-7)
    # zero blocks (the zero-initialised layer): the sparse branch exactly; and the drop threshold
    zero = orc.salad_fused_blockproj(q, k, v, 16, 8, rp, ci, 1, np.zeros_like(wb), s).reshape(B, H, N, d)
    assert np.array_equal(zero, o_s)
    drop = orc.salad_fused_blockproj(q, k, v, 16, 8, rp, ci, 1, wb, s, tau=0.5).reshape(B, H, N, d)
    assert np.array_equal(drop[0], o_s[0])
    np.testing.assert_allclose(drop[1], got[1], rtol=0, atol=0)
    # row selection
    sel = np.array([0, 17, N + 5, B * H * N - 1], dtype=np.int64)
    np.testing.assert_array_equal(orc.salad_fused_blockproj(q, k, v, 16, 8, rp, ci, 1, wb, s, sel=sel),
                                  got.reshape(-1, d)[sel])


# ----------------------------------------------------------------------------------------
# Linear branch with the rotary embedding (Sec. 4.1: the linear branch carries a 3-D rotary
# embedding; rotation in the numerator only, the normaliser un-rotated)

def _rotation_matrix(cs):
    """Dense d x d block-diagonal rotation of one token from its [d/2, 2] cosine/sine rows."""
    d = 2 * cs.shape[0]
    R = np.zeros((d, d))
    for i, (c, s) in enumerate(cs.astype(np.float64)):
        R[2 * i, 2 * i] = c;  R[2 * i, 2 * i + 1] = -s
        R[2 * i + 1, 2 * i] = s;  R[2 * i + 1, 2 * i + 1] = c
    return R


def _angles_table(ang):
    return np.stack([np.cos(ang), np.sin(ang)], axis=-1).astype(np.float32)


def test_rope_linear_hand_example():
    # d = 2 (one pair), two tokens with angles 0 and pi/2, eps = 0.
    #   keys   k0 = (1, 0), k1 = (0, 1); rotated: (1, 0) and R(pi/2)(0, 1) = (-1, 0)
    #   values v0 = (2, 3), v1 = (5, 7)
    #   query 0 = (1, 0), angle 0:    weights <(1,0),(1,0)> = 1 and <(1,0),(-1,0)> = -1, normaliser 1 + 0
    #                                 -> O_l = v0 - v1 = (-3, -4)
    #   query 1 = (0, 1), angle pi/2: rotated (-1, 0): weights -1 and 1, normaliser 0 + 1 -> v1 - v0 = (3, 4)
    q = np.array([[1.0, 0.0], [0.0, 1.0]], dtype=np.float32).reshape(1, 1, 2, 2)
    k = np.array([[1.0, 0.0], [0.0, 1.0]], dtype=np.float32).reshape(1, 1, 2, 2)
    v = np.array([[2.0, 3.0], [5.0, 7.0]], dtype=np.float32).reshape(1, 1, 2, 2)
    rope = np.array([[[1.0, 0.0]], [[0.0, 1.0]]], dtype=np.float32)      # cos, sin of 0 and pi/2
    o = orc.linear_attn_rope(q, k, v, rope, eps=0.0)
    np.testing.assert_allclose(o, [[-3.0, -4.0], [3.0, 4.0]], atol=1e-12)
    kv, z = orc.linear_state_rope(k, v, rope)
    np.testing.assert_allclose(kv[0, 0], [[2.0 - 5.0, 3.0 - 7.0], [0.0, 0.0]], atol=1e-12)
    np.testing.assert_allclose(z[0, 0], [1.0, 1.0], atol=1e-12)


def test_rope_linear_vs_explicit_quadratic_form():
    B, H, N, d = 1, 2, 37, 8
    q, k, v = rand_qkv(B, H, N, d, 41)
    rng = np.random.default_rng(5)
    rope = _angles_table(rng.uniform(-np.pi, np.pi, size=(N, d // 2)))
    eps = 1e-6
    got = orc.linear_attn_rope(q, k, v, rope, eps=eps).reshape(B, H, N, d)
    R = [_rotation_matrix(rope[n]) for n in range(N)]
    for h in range(H):
        fq = np.maximum(q[0, h].astype(np.float64), 0.0)
        fk = np.maximum(k[0, h].astype(np.float64), 0.0)
        qr = np.stack([R[n] @ fq[n] for n in range(N)])
        kr = np.stack([R[n] @ fk[n] for n in range(N)])
        w = qr @ kr.T                                   # [N, N] rotated similarities
        den = (fq @ fk.T).sum(axis=1) + eps             # un-rotated normaliser
        want = (w @ v[0, h].astype(np.float64)) / den[:, None]
        np.testing.assert_allclose(got[0, h], want, rtol=1e-10, atol=1e-12)


def test_rope_linear_special_cases():
    B, H, N, d = 2, 2, 50, 16
    q, k, v = rand_qkv(B, H, N, d, 43)
    # zero angles: the plain linear attention of Eq. 3
    ident = _angles_table(np.zeros((N, d // 2)))
    np.testing.assert_allclose(orc.linear_attn_rope(q, k, v, ident), orc.linear_attn(q, k, v), rtol=1e-12, atol=1e-14)
    kv0, z0 = orc.linear_state(k, v)
    kv1, z1 = orc.linear_state_rope(k, v, ident)
    np.testing.assert_allclose(kv1, kv0, rtol=1e-12); np.testing.assert_allclose(z1, z0, rtol=1e-12)
    # relative positions only: angle = position * frequency; moving every token by the same offset
    # changes nothing
    freq = 10000.0 ** (-np.arange(d // 2) / (d // 2))
    pos = np.arange(N, dtype=np.float64)
    a = orc.linear_attn_rope(q, k, v, _angles_table(pos[:, None] * freq[None, :]))
    b = orc.linear_attn_rope(q, k, v, _angles_table((pos[:, None] + 17.0) * freq[None, :]))
    np.testing.assert_allclose(a, b, rtol=1e-5, atol=1e-6)          # the tables are fp32
    assert np.abs(a - orc.linear_attn(q, k, v)).max() > 1e-2          # and the rotation does something
    # the normaliser ignores the rotation: the state's Z is the plain one for any table
    rng = np.random.default_rng(9)
    rope = _angles_table(rng.uniform(-np.pi, np.pi, size=(N, d // 2)))
    _, z2 = orc.linear_state_rope(k, v, rope)
    np.testing.assert_allclose(z2, z0, rtol=1e-12)
    # a rotation by pi flips the sign of the rotated keys and queries alike: numerator unchanged
    flip = _angles_table(np.full((N, d // 2), np.pi))
    np.testing.assert_allclose(orc.linear_attn_rope(q, k, v, flip), orc.linear_attn(q, k, v), rtol=1e-5, atol=1e-6)
    # row selection gives the same rows
    sel = np.array([0, 7, N * 3 + 11, B * H * N - 1], dtype=np.int64)
    full = orc.linear_attn_rope(q, k, v, rope)
    np.testing.assert_allclose(orc.linear_attn_rope(q, k, v, rope, sel=sel), full[sel], rtol=1e-12)


def test_rope_fused_pins():
    wl = wlmod.C1
    q, k, v = (t.float().numpy() for t in wlmod.make_qkv(wl))
    T, Hs, Ws = wl.grid
    rp, ci = orc.mask_build(T, Hs, Ws, wl.Bq, wl.Bk, wl.windows)
    lam, s = wlmod.make_scales(wl)
    sel = wlmod.sample_rows(wl, 64, seed=3)
    rope = orc.rope3d_table_vectorized(wl.grid, wl.d)
    # zero angles: Algorithm 1 as before
    ident = _angles_table(np.zeros((wl.N, wl.d // 2)))
    a = orc.salad_fused_rope(q, k, v, ident, wl.Bq, wl.Bk, rp, ci, wl.Hm, lam, s, sel=sel)
    b = orc.salad_fused(q, k, v, wl.Bq, wl.Bk, rp, ci, wl.Hm, lam, s, sel=sel)
    np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-14)
    # the sum of its parts
    o_s, _ = orc.sparse_attn(q, k, v, wl.Bq, wl.Bk, rp, ci, wl.Hm, sel=sel)
    o_l = orc.linear_attn_rope(q, k, v, rope, sel=sel)
    heads = (sel // wl.N) % wl.H
    want = o_s + (np.float64(s[0]) * lam.astype(np.float64)[heads])[:, None] * o_l
    got = orc.salad_fused_rope(q, k, v, rope, wl.Bq, wl.Bk, rp, ci, wl.Hm, lam, s, sel=sel)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-14)
    # dropped branch: the sparse output alone
    dropped = orc.salad_fused_rope(q, k, v, rope, wl.Bq, wl.Bk, rp, ci, wl.Hm, lam, s, tau=2.0, sel=sel)
    np.testing.assert_allclose(dropped, o_s, rtol=0, atol=0)


def test_rope3d_table_pins():
    grid, d = (3, 4, 5), 32
    r16 = orc.rope3d_table(grid, d)
    assert r16.dtype == np.float16                # the library's table dtype; 2^-11 relative rounding
    r = r16.astype(np.float64)
    N = 3 * 4 * 5
    assert r.shape == (N, d // 2, 2)
    np.testing.assert_allclose((r ** 2).sum(-1), 1.0, atol=2e-3)
    np.testing.assert_allclose(r[0, :, 0], 1.0); np.testing.assert_allclose(r[0, :, 1], 0.0)   # origin: no rotation
    p_hw = (d // 2) // 3; p_t = d // 2 - 2 * p_hw
    assert (p_t, p_hw) == (6, 5)
    n = lambda t, h, w: (t * 4 + h) * 5 + w
    # a step along w changes only the w pairs, by the pair's frequency
    np.testing.assert_allclose(r[n(1, 2, 3), :p_t + p_hw], r[n(1, 2, 4), :p_t + p_hw])
    ang = np.arctan2(r[n(0, 0, 1), p_t + p_hw:, 1], r[n(0, 0, 1), p_t + p_hw:, 0])
    np.testing.assert_allclose(ang, 10000.0 ** (-np.arange(p_hw) / p_hw), rtol=2e-2, atol=1e-3)
    # along h only the middle pairs, along t only the first p_t pairs
    np.testing.assert_allclose(r[n(1, 0, 3), :p_t], r[n(1, 3, 3), :p_t])
    np.testing.assert_allclose(r[n(1, 0, 3), p_t + p_hw:], r[n(1, 3, 3), p_t + p_hw:])
    np.testing.assert_allclose(r[n(0, 2, 3), p_t:], r[n(2, 2, 3), p_t:])
    ang_t = np.arctan2(r[n(1, 0, 0), :p_t, 1], r[n(1, 0, 0), :p_t, 0])
    np.testing.assert_allclose(ang_t, 10000.0 ** (-np.arange(p_t) / p_t), rtol=2e-2, atol=1e-3)
    # the first pair of every axis turns by one radian per position (frequency base**0 = 1)
    np.testing.assert_allclose(r[n(2, 3, 4), [0, p_t, p_t + p_hw], 0], np.cos([2.0, 3.0, 4.0]), atol=5e-4)
    np.testing.assert_allclose(r[n(2, 3, 4), [0, p_t, p_t + p_hw], 1], np.sin([2.0, 3.0, 4.0]), atol=5e-4)
    # rows on request, and the vectorised form the full-size tests use is the same table
    sel = [0, 7, 33, N - 1]
    assert np.array_equal(orc.rope3d_table(grid, d, tokens=sel).view(np.uint16), r16[sel].view(np.uint16))
    assert np.array_equal(orc.rope3d_table_vectorized(grid, d).view(np.uint16), r16.view(np.uint16))
    big = wlmod.C2.grid
    tok = np.random.default_rng(3).integers(0, wlmod.C2.N, size=200)
    assert np.array_equal(orc.rope3d_table_vectorized(big, 128)[tok].view(np.uint16),
                          orc.rope3d_table(big, 128, tokens=tok).view(np.uint16))
