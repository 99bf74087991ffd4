"""ctypes front end of the CPU oracle (``salad_oracle.c``).  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the CPU-baseline leg of the benchmark may import this
module.  It never touches the GPU library and the GPU library never touches it.

All array arguments are numpy arrays; Q, K, V are float32 arrays holding bf16-representable
values, shape [B, H, N, d].  Outputs are float64.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "salad_oracle.c")
_LIB = os.path.join(_HERE, "libsalad_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP only parallelises independent output rows)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-fvisibility=hidden",
             "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i32, i64, f64 = ctypes.c_int32, ctypes.c_int64, ctypes.c_double
        p = ctypes.c_void_p
        lib.oracle_mask_build.restype = i64
        lib.oracle_mask_build.argtypes = [i32] * 6 + [p, p, p, i64]
        lib.oracle_sparse_attn.restype = None
        lib.oracle_sparse_attn.argtypes = [p, p, p] + [i32] * 6 + [p, p, i32, f64, p, i64, p, p]
        lib.oracle_linear_state.restype = None
        lib.oracle_linear_state.argtypes = [p, p] + [i32] * 4 + [p, p]
        lib.oracle_linear_attn.restype = None
        lib.oracle_linear_attn.argtypes = [p, p, p] + [i32] * 4 + [f64, p, i64, p]
        lib.oracle_salad_fused.restype = None
        lib.oracle_salad_fused.argtypes = ([p, p, p] + [i32] * 6 + [p, p, i32, p, p, f64, f64,
                                                                    p, i64, p])
        lib.oracle_dynamic_scale.restype = None
        lib.oracle_dynamic_scale.argtypes = [p, p, f64, i32, i32, i32, p]
        lib.oracle_salad_fused_drop.restype = None
        lib.oracle_salad_fused_drop.argtypes = ([p, p, p] + [i32] * 6 + [p, p, i32, p, p, f64, f64, f64,
                                                                         p, i64, p])
        lib.oracle_salad_fused_blockproj.restype = None
        lib.oracle_salad_fused_blockproj.argtypes = ([p, p, p] + [i32] * 6 + [p, p, i32, p, p, f64, f64, f64,
                                                                               p, i64, p])
        lib.oracle_proj_combine.restype = None
        lib.oracle_proj_combine.argtypes = [p, p, p, p, p, i32, i32, i32, i32, p]
        lib.oracle_topk_mask.restype = None
        lib.oracle_topk_mask.argtypes = [p, p] + [i32] * 7 + [p, p]
        lib.oracle_linear_state_rope.restype = None
        lib.oracle_linear_state_rope.argtypes = [p, p, p] + [i32] * 4 + [p, p]
        lib.oracle_linear_attn_rope.restype = None
        lib.oracle_linear_attn_rope.argtypes = [p, p, p, p] + [i32] * 4 + [f64, p, i64, p]
        lib.oracle_salad_fused_rope.restype = None
        lib.oracle_salad_fused_rope.argtypes = ([p, p, p, p] + [i32] * 6 + [p, p, i32, p, p, f64, f64, f64,
                                                                            p, i64, p])
        lib.oracle_set_threads.restype = None
        lib.oracle_set_threads.argtypes = [i32]
        lib.oracle_max_threads.restype = i32
        lib.oracle_max_threads.argtypes = []
        _lib = lib
    return _lib


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a, a.ctypes.data


def _i32(a):
    a = np.ascontiguousarray(a, dtype=np.int32)
    return a, a.ctypes.data


def _sel(sel):
    if sel is None:
        return None, None, 0
    s = np.ascontiguousarray(sel, dtype=np.int64)
    return s, s.ctypes.data, int(s.size)


def num_threads() -> int:
    """Threads the oracle's parallel loops will use."""
    return int(_load().oracle_max_threads())


def use_all_cores() -> int:
    """Let the parallel loops use every core this process may run on, whatever OMP_NUM_THREADS says
    (launchers of multi-process jobs set it to 1).  Returns the thread count."""
    try:
        n = len(os.sched_getaffinity(0))
    except AttributeError:
        n = os.cpu_count() or 1
    _load().oracle_set_threads(n)
    return num_threads()


def mask_build(T, Hs, Ws, Bq, Bk, windows):
    """3-D sliding-window block mask -> (row_ptr[Hm*nQb+1], col_idx[nnz]) int32."""
    lib = _load()
    w, wp = _i32(np.asarray(windows).reshape(-1, 3))
    Hm = w.shape[0]
    N = T * Hs * Ws
    nQb = -(-N // Bq)
    row_ptr = np.zeros(Hm * nQb + 1, dtype=np.int32)
    nnz = lib.oracle_mask_build(T, Hs, Ws, Bq, Bk, Hm, wp, row_ptr.ctypes.data, None, 0)
    col_idx = np.zeros(max(nnz, 1), dtype=np.int32)
    lib.oracle_mask_build(T, Hs, Ws, Bq, Bk, Hm, wp, row_ptr.ctypes.data, col_idx.ctypes.data, nnz)
    return row_ptr, col_idx[:nnz]


def sparse_attn(q, k, v, Bq, Bk, row_ptr, col_idx, Hm, scale=None, sel=None):
    """Eq. 2 on the block mask.  Returns (O_s [rows, d] float64, lse [rows] float64)."""
    lib = _load()
    q, qp = _f32(q); k, kp = _f32(k); v, vp = _f32(v)
    B, H, N, d = q.shape
    rp, rpp = _i32(row_ptr); ci, cip = _i32(col_idx if len(col_idx) else np.zeros(1, np.int32))
    s, sp, nsel = _sel(sel)
    rows = nsel if s is not None else B * H * N
    o = np.empty((rows, d), dtype=np.float64)
    lse = np.empty(rows, dtype=np.float64)
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    lib.oracle_sparse_attn(qp, kp, vp, B, H, N, d, Bq, Bk, rpp, cip, Hm, float(scale),
                           sp, nsel, o.ctypes.data, lse.ctypes.data)
    return o, lse


def linear_state(k, v):
    """Returns (KV [B,H,d,d], Z [B,H,d]) float64."""
    lib = _load()
    k, kp = _f32(k); v, vp = _f32(v)
    B, H, N, d = k.shape
    kv = np.empty((B, H, d, d), dtype=np.float64)
    z = np.empty((B, H, d), dtype=np.float64)
    lib.oracle_linear_state(kp, vp, B, H, N, d, kv.ctypes.data, z.ctypes.data)
    return kv, z


def linear_attn(q, k, v, eps=1e-6, sel=None, state=None):
    """Eq. 3.  Returns O_l [rows, d] float64."""
    lib = _load()
    q, qp = _f32(q)
    B, H, N, d = q.shape
    kv, z = state if state is not None else linear_state(k, v)
    kv = np.ascontiguousarray(kv, dtype=np.float64); z = np.ascontiguousarray(z, dtype=np.float64)
    s, sp, nsel = _sel(sel)
    rows = nsel if s is not None else B * H * N
    o = np.empty((rows, d), dtype=np.float64)
    lib.oracle_linear_attn(qp, kv.ctypes.data, z.ctypes.data, B, H, N, d, float(eps),
                           sp, nsel, o.ctypes.data)
    return o


def salad_fused(q, k, v, Bq, Bk, row_ptr, col_idx, Hm, lambda_h, s_b, scale=None, eps=1e-6,
                sel=None):
    """Algorithm 1 residual integration: O_s + s_b * lambda_h * O_l.  [rows, d] float64."""
    lib = _load()
    q, qp = _f32(q); k, kp = _f32(k); v, vp = _f32(v)
    B, H, N, d = q.shape
    rp, rpp = _i32(row_ptr); ci, cip = _i32(col_idx if len(col_idx) else np.zeros(1, np.int32))
    lam = np.ascontiguousarray(lambda_h, dtype=np.float64); sb = np.ascontiguousarray(s_b, dtype=np.float64)
    assert lam.size == H and sb.size == B
    s, sp, nsel = _sel(sel)
    rows = nsel if s is not None else B * H * N
    o = np.empty((rows, d), dtype=np.float64)
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    lib.oracle_salad_fused(qp, kp, vp, B, H, N, d, Bq, Bk, rpp, cip, Hm, lam.ctypes.data,
                           sb.ctypes.data, float(scale), float(eps), sp, nsel, o.ctypes.data)
    return o


def dynamic_scale(x, w, bias=0.0):
    """Alg. 1 Level 2: s[b] = mean_n sigmoid(<x[b,n,:], w> + bias).  x [B,N,D], w [D] -> [B] float64."""
    lib = _load()
    x, xp = _f32(x); w, wp = _f32(w)
    B, N, D = x.shape
    assert w.size == D
    s = np.empty(B, dtype=np.float64)
    lib.oracle_dynamic_scale(xp, wp, float(bias), B, N, D, s.ctypes.data)
    return s


def salad_fused_drop(q, k, v, Bq, Bk, row_ptr, col_idx, Hm, lambda_h, s_b, tau, scale=None, eps=1e-6,
                     sel=None):
    """Fused output with branch dropping: the linear branch of batch item b is skipped when s_b < tau."""
    lib = _load()
    q, qp = _f32(q); k, kp = _f32(k); v, vp = _f32(v)
    B, H, N, d = q.shape
    rp, rpp = _i32(row_ptr); ci, cip = _i32(col_idx if len(col_idx) else np.zeros(1, np.int32))
    lam = np.ascontiguousarray(lambda_h, dtype=np.float64); sb = np.ascontiguousarray(s_b, dtype=np.float64)
    s, sp, nsel = _sel(sel)
    rows = nsel if s is not None else B * H * N
    o = np.empty((rows, d), dtype=np.float64)
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    lib.oracle_salad_fused_drop(qp, kp, vp, B, H, N, d, Bq, Bk, rpp, cip, Hm, lam.ctypes.data,
                                sb.ctypes.data, float(tau), float(scale), float(eps), sp, nsel, o.ctypes.data)
    return o


def salad_fused_blockproj(q, k, v, Bq, Bk, row_ptr, col_idx, Hm, w_blocks, s_b, tau=-np.inf, scale=None,
                          eps=1e-6, sel=None):
    """Algorithm 1 with one d x d projection block per head on the linear branch:
    O_s + [s_b >= tau] * s_b * W_h O_l, w_blocks [H, d, d] = W_h[c_out][a_in].  [rows, d] float64."""
    lib = _load()
    q, qp = _f32(q); k, kp = _f32(k); v, vp = _f32(v)
    B, H, N, d = q.shape
    rp, rpp = _i32(row_ptr); ci, cip = _i32(col_idx if len(col_idx) else np.zeros(1, np.int32))
    w, wp = _f32(w_blocks); assert w.shape == (H, d, d)
    sb = np.ascontiguousarray(s_b, dtype=np.float64); assert sb.size == B
    s, sp, nsel = _sel(sel)
    rows = nsel if s is not None else B * H * N
    o = np.empty((rows, d), dtype=np.float64)
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    lib.oracle_salad_fused_blockproj(qp, kp, vp, B, H, N, d, Bq, Bk, rpp, cip, Hm, wp, sb.ctypes.data,
                                     float(tau), float(scale), float(eps), sp, nsel, o.ctypes.data)
    return o


def topk_mask(q, k, Bq, Bk, topk, return_scores=False):
    """Dynamic Top-K block mask (Appendix A.1): per (batch, head) and query block the `topk` key blocks
    whose mean has the largest average similarity with the block's queries.
    Returns (row_ptr[B*H*nQb+1], col_idx[B*H*nQb*kk]) int32 (Hm = B*H), optionally the fp64 scores."""
    lib = _load()
    q, qp = _f32(q); k, kp = _f32(k)
    B, H, N, d = q.shape
    nQb, nKb = -(-N // Bq), -(-N // Bk)
    kk = min(int(topk), nKb)
    rows = B * H * nQb
    col_idx = np.zeros(rows * kk, dtype=np.int32)
    scores = np.zeros((B * H, nQb, nKb), dtype=np.float64) if return_scores else None
    lib.oracle_topk_mask(qp, kp, B, H, N, d, Bq, Bk, int(topk), col_idx.ctypes.data,
                         scores.ctypes.data if return_scores else None)
    row_ptr = (np.arange(rows + 1, dtype=np.int64) * kk).astype(np.int32)
    return (row_ptr, col_idx, scores) if return_scores else (row_ptr, col_idx)


def temporal_order(grid):
    """Appendix A.1 token permutation for heads with temporal locality: the flattening with time
    slowest, n = t*(Hs*Ws) + s, is replaced by one that groups tokens by spatial location, so that
    temporal neighbours are consecutive.  Returns perm with perm[m] = n: position m of the
    permuted sequence holds original token n, m = s*T + t."""
    T, Hs, Ws = grid
    S = Hs * Ws
    perm = np.empty(T * S, dtype=np.int64)
    for s in range(S):
        for t in range(T):
            perm[s * T + t] = t * S + s
    return perm


def permute_tokens(x, grid, head_flags, inverse=False):
    """x [B, H, N, d].  Heads with a non-zero flag are re-ordered along the token axis by
    temporal_order (forward: y[m] = x[perm[m]]; inverse: y[perm[m]] = x[m]); the others are copied."""
    x = np.asarray(x)
    perm = temporal_order(grid)
    y = x.copy()
    for h, flag in enumerate(head_flags):
        if flag:
            if inverse:
                y[:, h, perm] = x[:, h]
            else:
                y[:, h] = x[:, h, perm]
    return y


def proj_combine(o_s, o_l, w, s_b, bias=None):
    """Algorithm 1 with the full projection: O_s + s_b * Proj(O_l), Proj a D x D linear layer on the
    head-concatenated O_l (w[j_out, j_in], optional bias).  o_s, o_l [B,H,N,d] -> [B,H,N,d] float64."""
    lib = _load()
    o_s, sp = _f32(o_s); o_l, lp = _f32(o_l); w, wp = _f32(w)
    B, H, N, d = o_s.shape
    assert o_l.shape == o_s.shape and w.shape == (H * d, H * d)
    sb = np.ascontiguousarray(s_b, dtype=np.float64); assert sb.size == B
    if bias is not None:
        bias, bp = _f32(bias); assert bias.size == H * d
    else:
        bp = None
    out = np.empty((B, H, N, d), dtype=np.float64)
    lib.oracle_proj_combine(sp, lp, wp, bp, sb.ctypes.data, B, H, N, d, out.ctypes.data)
    return out


def _rope(rope, N, d):
    # any float dtype (the GPU library takes fp16): widened exactly to fp32 for the C routine
    r = np.ascontiguousarray(rope, dtype=np.float32)
    assert r.shape == (N, d // 2, 2), "rope is [N, d/2, 2]: cosine and sine of the angle of every token and channel pair"
    return r, r.ctypes.data


def linear_state_rope(k, v, rope):
    """Linear state with rotated keys: KV = sum_j (R_j ReLU(K_j))^T V_j, Z = sum_j ReLU(K_j).
    Returns (KV [B,H,d,d], Z [B,H,d]) float64."""
    lib = _load()
    k, kp = _f32(k); v, vp = _f32(v)
    B, H, N, d = k.shape
    r, rp = _rope(rope, N, d)
    kv = np.empty((B, H, d, d), dtype=np.float64)
    z = np.empty((B, H, d), dtype=np.float64)
    lib.oracle_linear_state_rope(kp, vp, rp, B, H, N, d, kv.ctypes.data, z.ctypes.data)
    return kv, z


def linear_attn_rope(q, k, v, rope, eps=1e-6, sel=None, state=None):
    """Eq. 3 with the rotary embedding in the numerator.  Returns O_l [rows, d] float64."""
    lib = _load()
    q, qp = _f32(q)
    B, H, N, d = q.shape
    r, rp = _rope(rope, N, d)
    kv, z = state if state is not None else linear_state_rope(k, v, rope)
    kv = np.ascontiguousarray(kv, dtype=np.float64); z = np.ascontiguousarray(z, dtype=np.float64)
    s, sp, nsel = _sel(sel)
    rows = nsel if s is not None else B * H * N
    o = np.empty((rows, d), dtype=np.float64)
    lib.oracle_linear_attn_rope(qp, rp, kv.ctypes.data, z.ctypes.data, B, H, N, d, float(eps),
                                sp, nsel, o.ctypes.data)
    return o


def salad_fused_rope(q, k, v, rope, Bq, Bk, row_ptr, col_idx, Hm, lambda_h, s_b, tau=-np.inf, scale=None,
                     eps=1e-6, sel=None):
    """Algorithm 1 with the rotary linear branch (and the drop threshold tau).  [rows, d] float64."""
    lib = _load()
    q, qp = _f32(q); k, kp = _f32(k); v, vp = _f32(v)
    B, H, N, d = q.shape
    r, rop = _rope(rope, N, d)
    rp, rpp = _i32(row_ptr); ci, cip = _i32(col_idx if len(col_idx) else np.zeros(1, np.int32))
    lam = np.ascontiguousarray(lambda_h, dtype=np.float64); sb = np.ascontiguousarray(s_b, dtype=np.float64)
    assert lam.size == H and sb.size == B
    s, sp, nsel = _sel(sel)
    rows = nsel if s is not None else B * H * N
    o = np.empty((rows, d), dtype=np.float64)
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    lib.oracle_salad_fused_rope(qp, kp, vp, rop, B, H, N, d, Bq, Bk, rpp, cip, Hm, lam.ctypes.data,
                                sb.ctypes.data, float(tau), float(scale), float(eps), sp, nsel, o.ctypes.data)
    return o


def rope3d_table(grid, d, base=10000.0, tokens=None):
    """Rotation table of a 3-D rotary position embedding for the tokens of a T x Hs x Ws latent grid
    (Sec. 4.1 says "3D"; the paper gives no layout, this one follows video DiTs of the Wan family):
    the d/2 channel pairs are shared out among the axes, floor(d/6) pairs each for h and w (in that order,
    after the t pairs) and the rest for t; pair j of an axis with P pairs turns by
        angle = position * base**(-j / P)
    for a token at that position along the axis; tokens are numbered with time slowest,
    n = (t*Hs + h)*Ws + w.  Angles, cosines and sines in float64, rounded once to float16 (the dtype of
    the GPU library's table).  Returns float16 [N, d/2, 2] = (cos, sin), or the rows of `tokens` only."""
    T, Hs, Ws = grid
    pairs = d // 2
    p_hw = pairs // 3
    p_t = pairs - 2 * p_hw
    tokens = range(T * Hs * Ws) if tokens is None else [int(n) for n in tokens]
    table = np.empty((len(tokens), pairs, 2), dtype=np.float16)
    for row, n in enumerate(tokens):
        pos = (n // (Hs * Ws), (n // Ws) % Hs, n % Ws)
        i = 0
        for axis, P in enumerate((p_t, p_hw, p_hw)):
            for j in range(P):
                angle = float(pos[axis]) * float(base) ** (-float(j) / P)
                table[row, i, 0] = np.float16(np.cos(angle))
                table[row, i, 1] = np.float16(np.sin(angle))
                i += 1
    return table


def rope3d_table_vectorized(grid, d: int, base: float = 10000.0) -> np.ndarray:
    """The table of rope3d_table computed with array operations instead of a loop over tokens and pairs,
    so that full-size tables (32 760 or 75 600 tokens) take milliseconds; the same float64 angles, rounded
    once to float16.  Pinned bit for bit to rope3d_table by the tests.  float16 [N, d/2, 2] = (cos, sin)."""
    T, Hs, Ws = grid
    pairs = d // 2
    p_hw = pairs // 3
    p_t = pairs - 2 * p_hw
    t, h, w = np.meshgrid(np.arange(T), np.arange(Hs), np.arange(Ws), indexing="ij")
    parts = []
    for pos, P in ((t, p_t), (h, p_hw), (w, p_hw)):
        freq = base ** (-np.arange(P, dtype=np.float64) / max(P, 1))
        parts.append(pos.reshape(-1, 1).astype(np.float64) * freq[None, :])
    ang = np.concatenate(parts, axis=1)                      # [N, d/2]
    return np.stack([np.cos(ang), np.sin(ang)], axis=-1).astype(np.float16)
