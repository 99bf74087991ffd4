"""ctypes binding of ``libsalad.so``: the same entry points as ``include/salad.h``.

The functions here only marshal arguments (tensor -> device pointer, sizes, the current
CUDA stream) and allocate outputs / workspace with torch when the caller does not pass
them.  Every step of the attention path runs inside the CUDA library; there is no other
implementation to fall back to: if the library is missing, importing this module fails.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsalad.so")

SALAD_OK = 0
SALAD_ERR_INVALID_ARG = -1
SALAD_ERR_UNSUPPORTED = -2
SALAD_ERR_WORKSPACE = -3
SALAD_ERR_CAPACITY = -4
SALAD_ERR_CUDA = -5
SALAD_ERR_TIMEOUT = -6
SALAD_ERR_BAD_MASK = -7

EXPORTS = ("salad_status_string", "salad_workspace_bytes", "salad_mask_build",
           "salad_sparse_attn_fwd", "salad_linear_attn_fwd", "salad_fused_fwd",
           "salad_set_profile_events", "salad_linear_attn_fwd_noalloc", "salad_fused_drop_fwd",
           "salad_dynamic_scale", "salad_topk_workspace_bytes", "salad_topk_mask_build", "salad_permute_tokens", "salad_proj_combine_fwd",
           "salad_selftest_bounded_wait", "salad_fused_rope_fwd", "salad_linear_attn_rope_fwd",
           "salad_rope3d_table_build", "salad_csr_validate", "salad_set_mask_validation",
           "salad_fused_proj_fwd", "salad_linear_state_fwd", "salad_fused_prepared_fwd",
           "salad_stswa_blocks", "salad_stswa_workspace_bytes", "salad_stswa_mask_build", "salad_fused_stswa_fwd")


class SaladError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where} failed: {status_string(code)} ({code})")


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} not found: build it with `python -m paper_2601_16515_b200.build` "
            "(there is no non-CUDA implementation to fall back to)")
    lib = ctypes.CDLL(LIB_PATH)
    i32, i64, f32, p, sz = ctypes.c_int, ctypes.c_int64, ctypes.c_float, ctypes.c_void_p, ctypes.c_size_t
    lib.salad_status_string.restype = ctypes.c_char_p
    lib.salad_status_string.argtypes = [i32]
    lib.salad_workspace_bytes.restype = sz
    lib.salad_workspace_bytes.argtypes = [i32] * 6
    lib.salad_mask_build.restype = i32
    lib.salad_mask_build.argtypes = [i32] * 6 + [p, p, p, i64, p, p]
    lib.salad_sparse_attn_fwd.restype = i32
    lib.salad_sparse_attn_fwd.argtypes = [p, p, p, p, p] + [i32] * 6 + [p, p, i32, f32, p, sz, p, p]
    lib.salad_linear_attn_fwd.restype = i32
    lib.salad_linear_attn_fwd.argtypes = [p, p, p, p, p, p] + [i32] * 4 + [f32, p, sz, p, p]
    lib.salad_fused_fwd.restype = i32
    lib.salad_fused_fwd.argtypes = [p, p, p, p] + [i32] * 6 + [p, p, i32, p, p, f32, f32, p, sz, p, p]
    lib.salad_linear_attn_fwd_noalloc.restype = i32
    lib.salad_linear_attn_fwd_noalloc.argtypes = [p, p, p, p, p, p] + [i32] * 4 + [f32, p, p]
    lib.salad_fused_drop_fwd.restype = i32
    lib.salad_fused_drop_fwd.argtypes = [p, p, p, p] + [i32] * 6 + [p, p, i32, p, p, f32, f32, f32, p, sz, p, p]
    lib.salad_dynamic_scale.restype = i32
    lib.salad_dynamic_scale.argtypes = [p, p, f32, i32, i32, i32, p, p, sz, p]
    lib.salad_topk_workspace_bytes.restype = sz
    lib.salad_topk_workspace_bytes.argtypes = [i32] * 6
    lib.salad_topk_mask_build.restype = i32
    lib.salad_topk_mask_build.argtypes = [p, p] + [i32] * 7 + [p, p, ctypes.c_int64, p, sz, p]
    lib.salad_permute_tokens.restype = i32
    lib.salad_permute_tokens.argtypes = [p, p] + [i32] * 7 + [p, i32, p]
    lib.salad_proj_combine_fwd.restype = i32
    lib.salad_proj_combine_fwd.argtypes = [p, p, p, p, p, p] + [i32] * 4 + [p, p]
    lib.salad_selftest_bounded_wait.restype = i32
    lib.salad_selftest_bounded_wait.argtypes = [p, p, p]
    lib.salad_fused_rope_fwd.restype = i32
    lib.salad_fused_rope_fwd.argtypes = [p, p, p, p] + [i32] * 6 + [p, p, i32, p, p, p, f32, f32, f32, p, sz, p, p]
    lib.salad_linear_attn_rope_fwd.restype = i32
    lib.salad_linear_attn_rope_fwd.argtypes = [p, p, p, p, p, p] + [i32] * 4 + [p, f32, p, sz, p, p]
    lib.salad_rope3d_table_build.restype = i32
    lib.salad_rope3d_table_build.argtypes = [i32, i32, i32, i32, f32, p, p]
    lib.salad_set_profile_events.restype = i32
    lib.salad_set_profile_events.argtypes = [p]
    lib.salad_fused_proj_fwd.restype = i32
    lib.salad_fused_proj_fwd.argtypes = [p, p, p, p] + [i32] * 6 + [p, p, i32, p, p, f32, f32, f32, p, sz, p, p]
    lib.salad_linear_state_fwd.restype = i32
    lib.salad_linear_state_fwd.argtypes = [p, p, p, p] + [i32] * 4 + [p, sz, p, p]
    lib.salad_fused_prepared_fwd.restype = i32
    lib.salad_fused_prepared_fwd.argtypes = [p, p, p, p] + [i32] * 6 + [p, p, i32, p, p, f32, f32, f32, p, sz, p, p]
    lib.salad_stswa_blocks.restype = i32
    lib.salad_stswa_blocks.argtypes = [i32, i32, i32, p, p, p, p]
    lib.salad_stswa_workspace_bytes.restype = sz
    lib.salad_stswa_workspace_bytes.argtypes = [i32] * 6
    lib.salad_stswa_mask_build.restype = i32
    lib.salad_stswa_mask_build.argtypes = [i32, i32, i32, i32, p, p, p, p, i64, p, p]
    lib.salad_fused_stswa_fwd.restype = i32
    lib.salad_fused_stswa_fwd.argtypes = [p, p, p, p] + [i32] * 7 + [p, p, p, p, p, f32, f32, f32, p, sz, p, p]
    lib.salad_csr_validate.restype = i32
    lib.salad_csr_validate.argtypes = [p, p, i64, i64, i32, p, p]
    lib.salad_set_mask_validation.restype = i32
    lib.salad_set_mask_validation.argtypes = [i64]
    return lib


_lib = _load()


def status_string(code: int) -> str:
    return _lib.salad_status_string(int(code)).decode()


def _check(rc: int, where: str):
    if rc != SALAD_OK:
        raise SaladError(rc, where)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _bf16_4d(name: str, t: torch.Tensor):
    if t.dtype != torch.bfloat16 or t.dim() != 4 or not t.is_contiguous() or not t.is_cuda:
        raise ValueError(f"{name} must be a contiguous CUDA bf16 tensor [B, H, N, d]")


def salad_workspace_bytes(B: int, H: int, N: int, d: int, Bq: int = 128, Bk: int = 64) -> int:
    return int(_lib.salad_workspace_bytes(B, H, N, d, Bq, Bk))


def alloc_workspace(B, H, N, d, Bq=128, Bk=64, device="cuda") -> torch.Tensor:
    n = salad_workspace_bytes(B, H, N, d, Bq, Bk)
    if n == 0:
        raise SaladError(SALAD_ERR_UNSUPPORTED, "salad_workspace_bytes")
    return torch.empty(n, dtype=torch.uint8, device=device)


def salad_mask_build(T: int, Hs: int, Ws: int, Bq: int, Bk: int,
                     windows: Sequence[Tuple[int, int, int]], device="cuda",
                     stream=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Sliding-window block mask -> (row_ptr int32 [Hm*nQb+1], col_idx int32 [nnz]) on device."""
    Hm = len(windows)
    flat = [int(x) for w in windows for x in w]
    h_win = (ctypes.c_int32 * max(1, len(flat)))(*flat)
    N = T * Hs * Ws
    nQb = -(-N // Bq)
    row_ptr = torch.empty(Hm * nQb + 1, dtype=torch.int32, device=device)
    nnz = ctypes.c_int64(-1)
    with torch.cuda.device(row_ptr.device):
        _check(_lib.salad_mask_build(T, Hs, Ws, Bq, Bk, Hm, h_win, _ptr(row_ptr), None, 0,
                                     ctypes.byref(nnz), _stream(stream)), "salad_mask_build")
        col_idx = torch.empty(max(1, nnz.value), dtype=torch.int32, device=device)
        _check(_lib.salad_mask_build(T, Hs, Ws, Bq, Bk, Hm, h_win, _ptr(row_ptr), _ptr(col_idx),
                                     col_idx.numel(), ctypes.byref(nnz), _stream(stream)), "salad_mask_build")
    return row_ptr, col_idx[:nnz.value]


def salad_csr_validate(row_ptr, col_idx, nKb: int, status=None, stream=None):
    """Checks CSR block lists (row_ptr int32 [rows+1], col_idx int32) against the library's contract.
    Returns the device status tensor: 0 = valid, SALAD_ERR_BAD_MASK = rejected (read it after a sync)."""
    _i32("row_ptr", row_ptr); _i32("col_idx", col_idx)
    if status is None:
        status = torch.zeros(1, dtype=torch.int32, device=row_ptr.device)
    with torch.cuda.device(row_ptr.device):
        _check(_lib.salad_csr_validate(_ptr(row_ptr), _ptr(col_idx), col_idx.numel(), row_ptr.numel() - 1, int(nKb),
                                       _ptr(status), _stream(stream)), "salad_csr_validate")
    return status


def salad_set_mask_validation(col_capacity: int = 0):
    """col_capacity > 0: the attention calls of this host thread validate their lists first (col_idx holding
    that many entries); 0: off."""
    _check(_lib.salad_set_mask_validation(int(col_capacity)), "salad_set_mask_validation")


def salad_set_profile_events(events=None):
    """events: None, or four torch.cuda.Event(enable_timing=True) / None entries:
    (state start, state stop, attention start, attention stop).  The events must have been
    recorded once (or otherwise materialised) so that they own a CUDA handle."""
    if events is None:
        _check(_lib.salad_set_profile_events(None), "salad_set_profile_events")
        return
    arr = (ctypes.c_void_p * 4)(*[None if e is None else e.cuda_event for e in events])
    _check(_lib.salad_set_profile_events(arr), "salad_set_profile_events")


def _common(q, k, v, Bq, Bk, workspace):
    for name, t in (("q", q), ("k", k), ("v", v)):
        _bf16_4d(name, t)
    if k.shape != q.shape or v.shape != q.shape:
        raise ValueError("q, k, v must have the same shape")
    B, H, N, d = q.shape
    if workspace is None:
        workspace = alloc_workspace(B, H, N, d, Bq, Bk, q.device)
    return B, H, N, d, workspace


def _i32(name, t):
    if t.dtype != torch.int32 or not t.is_cuda or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous CUDA int32 tensor")


def salad_sparse_attn_fwd(q, k, v, row_ptr, col_idx, Hm: int, Bq: int = 128, Bk: int = 64,
                          softmax_scale: float = 0.0, out=None, lse=None, workspace=None,
                          status=None, stream=None):
    """Block-sparse softmax attention.  Returns `out` (bf16 [B,H,N,d]); pass `lse` (fp32
    [B,H,N]) to receive the row log-sum-exp as well."""
    B, H, N, d, workspace = _common(q, k, v, Bq, Bk, workspace)
    _i32("row_ptr", row_ptr); _i32("col_idx", col_idx)
    if out is None:
        out = torch.empty_like(q)
    with torch.cuda.device(q.device):
        _check(_lib.salad_sparse_attn_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(lse), B, H, N, d, Bq, Bk,
                                          _ptr(row_ptr), _ptr(col_idx), Hm, float(softmax_scale),
                                          _ptr(workspace), workspace.numel(), _ptr(status), _stream(stream)),
               "salad_sparse_attn_fwd")
    return out


def salad_linear_attn_fwd(q, k, v, eps: float = 1e-6, out=None, kv_out=None, z_out=None,
                          workspace=None, status=None, stream=None):
    """ReLU linear attention.  Returns `out` (bf16 [B,H,N,d]); `kv_out` fp32 [B,H,d,d] and
    `z_out` fp32 [B,H,d] receive the state when given."""
    B, H, N, d, workspace = _common(q, k, v, 128, 64, workspace)
    if out is None:
        out = torch.empty_like(q)
    with torch.cuda.device(q.device):
        _check(_lib.salad_linear_attn_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(kv_out), _ptr(z_out),
                                          B, H, N, d, float(eps), _ptr(workspace), workspace.numel(),
                                          _ptr(status), _stream(stream)), "salad_linear_attn_fwd")
    return out


def _rope_table(rope, N, d):
    if (rope.dtype != torch.float16 or not rope.is_cuda or not rope.is_contiguous()
            or tuple(rope.shape) != (N, d // 2, 2)):
        raise ValueError(f"rope must be a contiguous CUDA fp16 tensor of shape [{N}, {d // 2}, 2] (cosine, sine)")
    return rope


def salad_rope3d_table_build(T: int, Hs: int, Ws: int, d: int, base: float = 10000.0, out=None, device=None,
                             stream=None):
    """fp16 rotation table [T*Hs*Ws, d/2, 2] of the 3-D rotary embedding of a latent grid, on the device."""
    if out is None:
        out = torch.empty((T * Hs * Ws, d // 2, 2), dtype=torch.float16, device=device or "cuda")
    _rope_table(out, T * Hs * Ws, d)
    with torch.cuda.device(out.device):
        _check(_lib.salad_rope3d_table_build(T, Hs, Ws, d, float(base), _ptr(out), _stream(stream)),
               "salad_rope3d_table_build")
    return out


def salad_linear_attn_rope_fwd(q, k, v, rope, eps: float = 1e-6, out=None, kv_out=None, z_out=None,
                               workspace=None, status=None, stream=None):
    """ReLU linear attention with a rotary position embedding in the numerator.  `rope` is the fp16
    table [N, d/2, 2] of cosines and sines per token and channel pair."""
    B, H, N, d, workspace = _common(q, k, v, 128, 64, workspace)
    _rope_table(rope, N, d)
    if out is None:
        out = torch.empty_like(q)
    with torch.cuda.device(q.device):
        _check(_lib.salad_linear_attn_rope_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(kv_out), _ptr(z_out),
                                               B, H, N, d, _ptr(rope), float(eps), _ptr(workspace),
                                               workspace.numel(), _ptr(status), _stream(stream)),
               "salad_linear_attn_rope_fwd")
    return out


def salad_fused_rope_fwd(q, k, v, row_ptr, col_idx, Hm: int, static_scale, dyn_scale, rope, Bq: int = 128,
                         Bk: int = 64, softmax_scale: float = 0.0, eps: float = 1e-6, out=None,
                         workspace=None, status=None, stream=None, drop_tau: Optional[float] = None):
    """salad_fused_fwd with the rotary linear branch (and, with `drop_tau`, branch dropping)."""
    B, H, N, d, workspace = _common(q, k, v, Bq, Bk, workspace)
    _i32("row_ptr", row_ptr); _i32("col_idx", col_idx)
    _rope_table(rope, N, d)
    for name, t, n in (("static_scale", static_scale, H), ("dyn_scale", dyn_scale, B)):
        if t.dtype != torch.float32 or not t.is_cuda or t.numel() != n or not t.is_contiguous():
            raise ValueError(f"{name} must be a contiguous CUDA fp32 tensor with {n} elements")
    if out is None:
        out = torch.empty_like(q)
    tau = float("-inf") if drop_tau is None else float(drop_tau)
    with torch.cuda.device(q.device):
        _check(_lib.salad_fused_rope_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, H, N, d, Bq, Bk,
                                         _ptr(row_ptr), _ptr(col_idx), Hm, _ptr(static_scale), _ptr(dyn_scale),
                                         _ptr(rope), tau, float(softmax_scale), float(eps), _ptr(workspace),
                                         workspace.numel(), _ptr(status), _stream(stream)),
               "salad_fused_rope_fwd")
    return out


def salad_linear_state_fwd(k, v, workspace, kv_out=None, z_out=None, status=None, stream=None):
    """The linear state (KV, Z of Eq. 3) of K, V into `workspace`, for a later salad_fused_prepared_fwd call on
    the same workspace; kv_out fp32 [B,H,d,d] and z_out fp32 [B,H,d] receive copies when given."""
    for name, t in (("k", k), ("v", v)):
        _bf16_4d(name, t)
    if k.shape != v.shape:
        raise ValueError("k and v must have the same shape")
    B, H, N, d = k.shape
    with torch.cuda.device(k.device):
        _check(_lib.salad_linear_state_fwd(_ptr(k), _ptr(v), _ptr(kv_out), _ptr(z_out), B, H, N, d, _ptr(workspace),
                                           workspace.numel(), _ptr(status), _stream(stream)), "salad_linear_state_fwd")
    return workspace


def salad_fused_prepared_fwd(q, k, v, row_ptr, col_idx, Hm: int, static_scale, dyn_scale, workspace, Bq: int = 128,
                             Bk: int = 64, softmax_scale: float = 0.0, eps: float = 1e-6, out=None, status=None,
                             stream=None, drop_tau: Optional[float] = None):
    """salad_fused_fwd on a workspace that already holds the linear state (salad_linear_state_fwd)."""
    B, H, N, d, workspace = _common(q, k, v, Bq, Bk, workspace)
    _i32("row_ptr", row_ptr); _i32("col_idx", col_idx)
    for name, t, n in (("static_scale", static_scale, H), ("dyn_scale", dyn_scale, B)):
        if t.dtype != torch.float32 or not t.is_cuda or t.numel() != n or not t.is_contiguous():
            raise ValueError(f"{name} must be a contiguous CUDA fp32 tensor with {n} elements")
    if out is None:
        out = torch.empty_like(q)
    tau = float("-inf") if drop_tau is None else float(drop_tau)
    with torch.cuda.device(q.device):
        _check(_lib.salad_fused_prepared_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, H, N, d, Bq, Bk,
                                             _ptr(row_ptr), _ptr(col_idx), Hm, _ptr(static_scale), _ptr(dyn_scale), tau,
                                             float(softmax_scale), float(eps), _ptr(workspace), workspace.numel(),
                                             _ptr(status), _stream(stream)), "salad_fused_prepared_fwd")
    return out


def salad_fused_proj_fwd(q, k, v, row_ptr, col_idx, Hm: int, proj_blocks, dyn_scale, Bq: int = 128, Bk: int = 64,
                         softmax_scale: float = 0.0, eps: float = 1e-6, out=None, workspace=None, status=None,
                         stream=None, drop_tau: Optional[float] = None):
    """O = O_sparse + dyn_scale[b] * W_h O_linear with one d x d projection block per head
    (proj_blocks bf16 [H, d, d], W_h[c_out][a_in]), one bf16 write."""
    B, H, N, d, workspace = _common(q, k, v, Bq, Bk, workspace)
    _i32("row_ptr", row_ptr); _i32("col_idx", col_idx)
    if (proj_blocks.dtype != torch.bfloat16 or not proj_blocks.is_cuda or not proj_blocks.is_contiguous()
            or tuple(proj_blocks.shape) != (H, d, d)):
        raise ValueError(f"proj_blocks must be a contiguous CUDA bf16 tensor [{H}, {d}, {d}]")
    if dyn_scale.dtype != torch.float32 or not dyn_scale.is_cuda or dyn_scale.numel() != B or not dyn_scale.is_contiguous():
        raise ValueError(f"dyn_scale must be a contiguous CUDA fp32 tensor with {B} elements")
    if out is None:
        out = torch.empty_like(q)
    tau = float("-inf") if drop_tau is None else float(drop_tau)
    with torch.cuda.device(q.device):
        _check(_lib.salad_fused_proj_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, H, N, d, Bq, Bk,
                                         _ptr(row_ptr), _ptr(col_idx), Hm, _ptr(proj_blocks), _ptr(dyn_scale), tau,
                                         float(softmax_scale), float(eps), _ptr(workspace), workspace.numel(),
                                         _ptr(status), _stream(stream)), "salad_fused_proj_fwd")
    return out


NOALLOC_MAX_HEADS = 16


def salad_linear_attn_fwd_noalloc(q, k, v, eps: float = 1e-6, out=None, kv_out=None, z_out=None,
                                  status=None, stream=None):
    """ReLU linear attention without a workspace, for hosts that must not allocate device
    memory when attention runs (fixed memory pools, capture/replay, real-time loops).  The
    scratch is a fixed array inside the library (B*H <= 16, d in {64, 128}); calls on one
    device share it and must not overlap on the GPU.  Pass `out` to avoid the one output
    allocation this Python wrapper would otherwise make; the C entry point allocates nothing."""
    for name, t in (("q", q), ("k", k), ("v", v)):
        _bf16_4d(name, t)
    if k.shape != q.shape or v.shape != q.shape:
        raise ValueError("q, k, v must have the same shape")
    B, H, N, d = q.shape
    if out is None:
        out = torch.empty_like(q)
    with torch.cuda.device(q.device):
        _check(_lib.salad_linear_attn_fwd_noalloc(_ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(kv_out), _ptr(z_out),
                                                  B, H, N, d, float(eps), _ptr(status), _stream(stream)),
               "salad_linear_attn_fwd_noalloc")
    return out


def salad_topk_mask_build(q, k, topk: int, Bq: int = 128, Bk: int = 64, row_ptr=None, col_idx=None,
                          workspace=None, stream=None):
    """Top-K block mask of every (batch, head): returns (row_ptr, col_idx) int32 device tensors, to be
    passed to the attention calls with Hm = B*H."""
    for name, t in (("q", q), ("k", k)):
        _bf16_4d(name, t)
    if q.shape != k.shape:
        raise ValueError("q and k must have the same shape")
    B, H, N, d = q.shape
    nQb, nKb = -(-N // Bq), -(-N // Bk)
    kk = min(int(topk), nKb)
    rows = B * H * nQb
    if row_ptr is None:
        row_ptr = torch.empty(rows + 1, dtype=torch.int32, device=q.device)
    if col_idx is None:
        col_idx = torch.empty(max(rows * kk, 1), dtype=torch.int32, device=q.device)
    _i32("row_ptr", row_ptr); _i32("col_idx", col_idx)
    if workspace is None:
        nbytes = int(_lib.salad_topk_workspace_bytes(B, H, N, d, Bq, Bk))
        workspace = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=q.device)
    with torch.cuda.device(q.device):
        _check(_lib.salad_topk_mask_build(_ptr(q), _ptr(k), B, H, N, d, Bq, Bk, int(topk), _ptr(row_ptr),
                                          _ptr(col_idx), col_idx.numel(), _ptr(workspace), workspace.numel(),
                                          _stream(stream)), "salad_topk_mask_build")
    return row_ptr, col_idx[:rows * kk]


def salad_permute_tokens(x, grid, head_flags, inverse: bool = False, out=None, stream=None):
    """Re-order the tokens of the flagged heads from time-slowest to grouped-by-spatial-location order
    (inverse=True: back).  x bf16 [B,H,N,d]; grid = (T, Hs, Ws); head_flags: H ints."""
    _bf16_4d("x", x)
    B, H, N, d = x.shape
    T, Hs, Ws = grid
    flags = (ctypes.c_int32 * H)(*[int(bool(f)) for f in head_flags])
    if len(head_flags) != H:
        raise ValueError("head_flags must have one entry per head")
    if out is None:
        out = torch.empty_like(x)
    with torch.cuda.device(x.device):
        _check(_lib.salad_permute_tokens(_ptr(x), _ptr(out), B, H, N, d, T, Hs, Ws, flags, int(bool(inverse)),
                                         _stream(stream)), "salad_permute_tokens")
    return out


def salad_stswa_blocks(grid):
    """Block geometry of salad_fused_stswa_fwd on a (T, Hs, Ws) grid: (list rows per head, spatial positions
    per query block, per key block, key blocks of a temporal head)."""
    T, Hs, Ws = grid
    vals = [ctypes.c_int32(0) for _ in range(4)]
    _check(_lib.salad_stswa_blocks(T, Hs, Ws, *[ctypes.byref(x) for x in vals]), "salad_stswa_blocks")
    return tuple(int(x.value) for x in vals)


def salad_stswa_mask_build(grid, head_flags, windows, device="cuda", stream=None):
    """1-D sliding-window lists for salad_fused_stswa_fwd: windows[h] is the half-width of head h's window in
    tokens of its own order (grouped by spatial position when head_flags[h]).  Returns (row_ptr, col_idx)."""
    T, Hs, Ws = grid
    H = len(head_flags)
    rows = salad_stswa_blocks(grid)[0]
    flags = (ctypes.c_int32 * H)(*[int(bool(f)) for f in head_flags])
    win = (ctypes.c_int32 * H)(*[int(w) for w in windows])
    row_ptr = torch.empty(H * rows + 1, dtype=torch.int32, device=device)
    nnz = ctypes.c_int64(-1)
    with torch.cuda.device(row_ptr.device):
        _check(_lib.salad_stswa_mask_build(T, Hs, Ws, H, flags, win, _ptr(row_ptr), None, 0, ctypes.byref(nnz),
                                           _stream(stream)), "salad_stswa_mask_build")
        col_idx = torch.empty(max(1, nnz.value), dtype=torch.int32, device=device)
        _check(_lib.salad_stswa_mask_build(T, Hs, Ws, H, flags, win, _ptr(row_ptr), _ptr(col_idx), col_idx.numel(),
                                           ctypes.byref(nnz), _stream(stream)), "salad_stswa_mask_build")
    return row_ptr, col_idx[:nnz.value]


def salad_fused_stswa_fwd(q, k, v, grid, head_flags, row_ptr, col_idx, static_scale, dyn_scale, softmax_scale: float = 0.0,
                          eps: float = 1e-6, out=None, workspace=None, status=None, stream=None,
                          drop_tau: Optional[float] = None):
    """The fused call with the paper's ST-SWA: flagged heads take their tokens grouped by spatial position through
    the loads and stores themselves (no permutation pass); lists from salad_stswa_mask_build."""
    for name, t in (("q", q), ("k", k), ("v", v)):
        _bf16_4d(name, t)
    if k.shape != q.shape or v.shape != q.shape:
        raise ValueError("q, k, v must have the same shape")
    B, H, N, d = q.shape
    T, Hs, Ws = grid
    if len(head_flags) != H:
        raise ValueError("head_flags must have one entry per head")
    _i32("row_ptr", row_ptr); _i32("col_idx", col_idx)
    for name, t, n in (("static_scale", static_scale, H), ("dyn_scale", dyn_scale, B)):
        if t.dtype != torch.float32 or not t.is_cuda or t.numel() != n or not t.is_contiguous():
            raise ValueError(f"{name} must be a contiguous CUDA fp32 tensor with {n} elements")
    flags = (ctypes.c_int32 * H)(*[int(bool(f)) for f in head_flags])
    if workspace is None:
        nbytes = int(_lib.salad_stswa_workspace_bytes(B, H, T, Hs, Ws, d))
        if nbytes == 0:
            raise SaladError(SALAD_ERR_UNSUPPORTED, "salad_stswa_workspace_bytes")
        workspace = torch.empty(nbytes, dtype=torch.uint8, device=q.device)
    if out is None:
        out = torch.empty_like(q)
    tau = float("-inf") if drop_tau is None else float(drop_tau)
    with torch.cuda.device(q.device):
        _check(_lib.salad_fused_stswa_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, H, N, d, T, Hs, Ws, flags,
                                          _ptr(row_ptr), _ptr(col_idx), _ptr(static_scale), _ptr(dyn_scale), tau,
                                          float(softmax_scale), float(eps), _ptr(workspace), workspace.numel(),
                                          _ptr(status), _stream(stream)), "salad_fused_stswa_fwd")
    return out


def salad_proj_combine_fwd(o_s, o_l, w, dyn_scale=None, bias=None, out=None, status=None, stream=None):
    """out = O_s + dyn_scale[b] * (concat_heads(O_l) @ w.T + bias), all [B,H,N,d] bf16; w bf16 [D,D]."""
    _bf16_4d("o_s", o_s); _bf16_4d("o_l", o_l)
    if o_s.shape != o_l.shape:
        raise ValueError("o_s and o_l must have the same shape")
    B, H, N, d = o_s.shape
    D = H * d
    if w.dtype != torch.bfloat16 or not w.is_cuda or not w.is_contiguous() or tuple(w.shape) != (D, D):
        raise ValueError("w must be a contiguous CUDA bf16 tensor [H*d, H*d]")
    for name, t, n in (("dyn_scale", dyn_scale, B), ("bias", bias, D)):
        if t is not None and (t.dtype != torch.float32 or not t.is_cuda or t.numel() != n or not t.is_contiguous()):
            raise ValueError(f"{name} must be a contiguous CUDA fp32 tensor with {n} elements")
    if out is None:
        out = torch.empty_like(o_s)
    with torch.cuda.device(o_s.device):
        _check(_lib.salad_proj_combine_fwd(_ptr(o_s), _ptr(o_l), _ptr(w), _ptr(bias), _ptr(dyn_scale), _ptr(out),
                                           B, H, N, d, _ptr(status), _stream(stream)), "salad_proj_combine_fwd")
    return out


def salad_selftest_bounded_wait(stream=None):
    """Runs the bounded-wait self-test kernel; returns (status, waited_ns) device tensors."""
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    waited = torch.zeros(1, dtype=torch.int64, device="cuda")
    _check(_lib.salad_selftest_bounded_wait(_ptr(status), _ptr(waited), _stream(stream)), "salad_selftest_bounded_wait")
    return status, waited


DYN_SCALE_WS_BYTES = 8192


def salad_dynamic_scale(x, w, bias: float = 0.0, out=None, workspace=None, stream=None):
    """s[b] = mean over tokens of sigmoid(<x[b,n,:], w> + bias).  x bf16 [B,N,D], w fp32 [D] -> fp32 [B]."""
    if x.dtype != torch.bfloat16 or x.dim() != 3 or not x.is_contiguous() or not x.is_cuda:
        raise ValueError("x must be a contiguous CUDA bf16 tensor [B, N, D]")
    B, N, D = x.shape
    if w.dtype != torch.float32 or not w.is_cuda or w.numel() != D or not w.is_contiguous():
        raise ValueError("w must be a contiguous CUDA fp32 tensor with D elements")
    if out is None:
        out = torch.empty(B, dtype=torch.float32, device=x.device)
    if workspace is None:
        workspace = torch.empty(DYN_SCALE_WS_BYTES, dtype=torch.uint8, device=x.device)
    with torch.cuda.device(x.device):
        _check(_lib.salad_dynamic_scale(_ptr(x), _ptr(w), float(bias), B, N, D, _ptr(out), _ptr(workspace),
                                        workspace.numel(), _stream(stream)), "salad_dynamic_scale")
    return out


def salad_fused_fwd(q, k, v, row_ptr, col_idx, Hm: int, static_scale, dyn_scale, Bq: int = 128,
                    Bk: int = 64, softmax_scale: float = 0.0, eps: float = 1e-6, out=None,
                    workspace=None, status=None, stream=None, drop_tau: Optional[float] = None):
    """O = O_sparse + dyn_scale[b] * static_scale[h] * O_linear, one bf16 write.  With `drop_tau`
    the linear branch of batch items whose dyn_scale is below it is skipped (salad_fused_drop_fwd)."""
    B, H, N, d, workspace = _common(q, k, v, Bq, Bk, workspace)
    _i32("row_ptr", row_ptr); _i32("col_idx", col_idx)
    for name, t, n in (("static_scale", static_scale, H), ("dyn_scale", dyn_scale, B)):
        if t.dtype != torch.float32 or not t.is_cuda or t.numel() != n or not t.is_contiguous():
            raise ValueError(f"{name} must be a contiguous CUDA fp32 tensor with {n} elements")
    if out is None:
        out = torch.empty_like(q)
    with torch.cuda.device(q.device):
        if drop_tau is None:
            _check(_lib.salad_fused_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, H, N, d, Bq, Bk,
                                        _ptr(row_ptr), _ptr(col_idx), Hm, _ptr(static_scale), _ptr(dyn_scale),
                                        float(softmax_scale), float(eps), _ptr(workspace), workspace.numel(),
                                        _ptr(status), _stream(stream)), "salad_fused_fwd")
        else:
            _check(_lib.salad_fused_drop_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, H, N, d, Bq, Bk,
                                             _ptr(row_ptr), _ptr(col_idx), Hm, _ptr(static_scale), _ptr(dyn_scale),
                                             float(drop_tau), float(softmax_scale), float(eps), _ptr(workspace),
                                             workspace.numel(), _ptr(status), _stream(stream)),
                   "salad_fused_drop_fwd")
    return out
