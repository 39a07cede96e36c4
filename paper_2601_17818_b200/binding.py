"""Thin ctypes binding of ``libvitcop.so`` -- same entry-point names as ``include/vitcop.h``.

Argument marshalling only: every function takes torch CUDA tensors (or ``None``), passes their
``data_ptr()`` and the current CUDA stream to the C ABI and raises ``VitcopError`` on a non-zero
status.  No arithmetic of the method happens here, and there is no fallback: if the shared
library is missing or fails to load, importing the functions raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libvitcop.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_BUDGET, ERR_CUDA, ERR_TIMEOUT = range(7)
(OP_FILTER, OP_KNORM, OP_SELECT, OP_COMPACT, OP_PRUNE_STEP, OP_SIMILARITY, OP_SALIENCY, OP_MERGE, OP_COLLAB_STEP,
 OP_KPROJ) = range(10)
MAX_VISUAL_TOKENS = 16384

EXPORTS = [
    "vitcop_status_string", "vitcop_last_cuda_error", "vitcop_workspace_bytes", "vitcop_poll_status",
    "vitcop_redundancy_filter", "vitcop_similarity_rows", "vitcop_knorm_score", "vitcop_select",
    "vitcop_compact_kv", "vitcop_prune_step", "vitcop_kernel_timing_begin", "vitcop_kernel_timing_end",
    "vitcop_prune_step_static", "vitcop_merge_clusters", "vitcop_cls_saliency", "vitcop_stage_count",
    "vitcop_flops_layer", "vitcop_visual_tokens_at_layer", "vitcop_flops_total", "vitcop_cr_int",
    "vitcop_collaborative_step", "vitcop_set_wait_limit", "vitcop_kproj_knorm",
]


class VitcopError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().vitcop_status_string(status).decode()
        if status == ERR_CUDA:
            msg += f" (cudaError {lib().vitcop_last_cuda_error()})"
        super().__init__(f"{where}: {msg} [status {status}]")


class FilterParams(C.Structure):
    _fields_ = [("metric", C.c_int), ("d_c", C.c_float), ("tau", C.c_float), ("alpha", C.c_double),
                ("n_centers", C.c_int)]


class KernelTime(C.Structure):
    _fields_ = [("name", C.c_char * 48), ("launches", C.c_int), ("total_ms", C.c_float)]


class SelectParams(C.Structure):
    _fields_ = [("mode", C.c_int), ("largest", C.c_int), ("budget", C.c_int)]


_lib: Optional[C.CDLL] = None


def lib() -> C.CDLL:
    """Loads the shared library (once).  Fails loudly when it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2601_17818_b200.build` first")
        L = C.CDLL(LIB_PATH)
        L.vitcop_status_string.restype = C.c_char_p
        L.vitcop_status_string.argtypes = [C.c_int]
        L.vitcop_last_cuda_error.restype = C.c_int
        vp, i32, i64, sz = C.c_void_p, C.c_int, C.c_int64, C.c_size_t
        L.vitcop_workspace_bytes.argtypes = [i32] * 8 + [C.POINTER(sz)]
        L.vitcop_poll_status.argtypes = [vp, vp, C.POINTER(C.c_int)]
        L.vitcop_redundancy_filter.argtypes = [vp, vp, i32, i32, i32, C.POINTER(FilterParams), vp, vp, vp, vp, vp,
                                               vp, sz, vp]
        L.vitcop_similarity_rows.argtypes = [vp, i32, i32, i32, i32, i32, i32, vp, vp, sz, vp]
        L.vitcop_knorm_score.argtypes = [vp, i32, i32, i32, i32, i64, i64, i64, i32, vp, i32, vp, i32, vp]
        L.vitcop_select.argtypes = [vp, vp, i32, vp, i32, i32, C.POINTER(SelectParams), vp, i32, vp, vp, vp, sz, vp]
        L.vitcop_compact_kv.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, vp, i32, vp, i32, vp, i32, vp,
                                        vp, vp, vp, i32, vp, vp, vp]
        L.vitcop_prune_step.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, vp, i32, vp, i32, i32, vp, i32,
                                        vp, vp, vp, i32, vp, vp, vp, vp, vp, vp, sz, vp]
        L.vitcop_prune_step_static.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, vp, i32, vp, i32, i32, vp, i32,
                                               vp, vp, vp, i32, vp, vp, vp, vp, vp, vp]
        L.vitcop_merge_clusters.argtypes = [vp, i32, i32, i32, i32, vp, i32, i32, vp, vp, vp, vp, vp, vp, vp, i32, vp, sz,
                                            vp]
        L.vitcop_cls_saliency.argtypes = [vp, vp, i32, i32, i32, i32, C.c_float, vp, vp, vp, sz, vp]
        f64 = C.c_double
        L.vitcop_stage_count.argtypes = [i32, f64]
        L.vitcop_flops_layer.argtypes = [f64, f64]
        L.vitcop_flops_layer.restype = f64
        L.vitcop_visual_tokens_at_layer.argtypes = [i32, f64, f64, f64, f64, i32, i32]
        L.vitcop_visual_tokens_at_layer.restype = f64
        L.vitcop_flops_total.argtypes = [f64, f64, f64, f64, f64, f64, i32, i32, i32]
        L.vitcop_flops_total.restype = f64
        L.vitcop_cr_int.argtypes = [f64, f64, f64, i32, i32, i32]
        L.vitcop_cr_int.restype = f64
        L.vitcop_collaborative_step.argtypes = [vp, vp, i32, C.POINTER(FilterParams), vp, vp, vp, i32, i32, i32, i32,
                                                i32, i32, i32, i32, vp, vp, vp, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp,
                                                vp, vp, sz, vp]
        L.vitcop_set_wait_limit.argtypes = [C.c_ulonglong, i32]
        L.vitcop_kproj_knorm.argtypes = [vp, vp, i32, i32, i32, i32, i32, vp, vp, vp, i32, vp, i32, i32, vp, vp, sz, vp]
        L.vitcop_kernel_timing_begin.argtypes = []
        L.vitcop_kernel_timing_end.argtypes = [C.POINTER(KernelTime), i32, C.POINTER(C.c_int)]
        for name in EXPORTS:
            getattr(L, name)
        _lib = L
    return _lib


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("expected a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError("expected a contiguous tensor")
    return C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(status: int, where: str):
    if status != OK:
        raise VitcopError(status, where)


def _vis(vis_len):
    """(device pointer or None, uniform length) from an int or an int32 CUDA tensor."""
    if isinstance(vis_len, torch.Tensor):
        assert vis_len.dtype == torch.int32
        return _ptr(vis_len), 0
    return None, int(vis_len)


# ----------------------------------------------------------------------------------------------
def vitcop_workspace_bytes(op: int, B=0, H=0, N=0, d=0, Nv=0, D=0, Dh=0) -> int:
    out = C.c_size_t(0)
    _check(lib().vitcop_workspace_bytes(op, B, H, N, d, Nv, D, Dh, C.byref(out)), "vitcop_workspace_bytes")
    return int(out.value)


def alloc_workspace(op: int, device="cuda", **dims) -> torch.Tensor:
    """A uint8 CUDA tensor large enough for ``op`` (torch allocations are at least 256-byte aligned)."""
    return torch.empty(max(vitcop_workspace_bytes(op, **dims), 256), dtype=torch.uint8, device=device)


def vitcop_poll_status(workspace: torch.Tensor) -> int:
    v = C.c_int(0)
    _check(lib().vitcop_poll_status(_ptr(workspace), _stream(), C.byref(v)), "vitcop_poll_status")
    return int(v.value)


def vitcop_knorm_score(K: torch.Tensor, vis_start: int, vis_len, score: torch.Tensor) -> torch.Tensor:
    """K bf16 [B,H,N,d] (last dim contiguous, arbitrary leading strides) -> score fp32 [B, Nv_cap]."""
    assert K.dtype == torch.bfloat16 and score.dtype == torch.float32 and K.dim() == 4 and K.stride(3) == 1
    B, H, N, d = K.shape
    vp, vu = _vis(vis_len)
    rc = lib().vitcop_knorm_score(C.c_void_p(K.data_ptr()), B, H, N, d, K.stride(0), K.stride(1), K.stride(2),
                                  vis_start, vp, vu, _ptr(score), score.shape[1], _stream())
    _check(rc, "vitcop_knorm_score")
    return score


def vitcop_select(score: torch.Tensor, vis_len, budget: int, keep_idx: torch.Tensor, n_keep: torch.Tensor,
                  workspace: torch.Tensor, label: Optional[torch.Tensor] = None, largest: bool = False,
                  keep_mask: Optional[torch.Tensor] = None, mode: Optional[int] = None):
    assert score.dtype == torch.float32 and keep_idx.dtype == torch.int32 and n_keep.dtype == torch.int32
    B, Nv_cap = score.shape
    p = SelectParams((1 if label is not None else 0) if mode is None else mode, int(largest), int(budget))
    vp, vu = _vis(vis_len)
    rc = lib().vitcop_select(_ptr(score), _ptr(label), B, vp, vu, Nv_cap, C.byref(p), _ptr(keep_idx),
                             keep_idx.shape[1], _ptr(n_keep), _ptr(keep_mask), _ptr(workspace), workspace.numel(),
                             _stream())
    _check(rc, "vitcop_select")
    return keep_idx, n_keep


def vitcop_compact_kv(hidden, K, V, vis_start: int, vis_len, keep_idx, n_keep, hidden_out, K_out, V_out,
                      out_len: torch.Tensor, kept_pos=None, seq_len=None):
    ref = K if K is not None else V
    if ref is not None:
        B, H, N, d = ref.shape
        Ncap = (K_out if K_out is not None else V_out).shape[2]
    else:
        B, N, _ = hidden.shape
        H, d = 0, 0
        Ncap = hidden_out.shape[1]
    Dh = hidden.shape[2] if hidden is not None else 0
    vp, vu = _vis(vis_len)
    rc = lib().vitcop_compact_kv(_ptr(hidden), _ptr(K), _ptr(V), B, H, N, d, Dh, _ptr(seq_len), vis_start, vp, vu,
                                 _ptr(keep_idx), keep_idx.shape[1], _ptr(n_keep), _ptr(hidden_out), _ptr(K_out),
                                 _ptr(V_out), Ncap, _ptr(kept_pos), _ptr(out_len), _stream())
    _check(rc, "vitcop_compact_kv")
    return out_len


def vitcop_prune_step(hidden, K, V, vis_start: int, vis_len, Nv_cap: int, budget: int, hidden_out, K_out, V_out,
                      out_len, workspace, label=None, kept_pos=None, seq_len=None, score_out=None,
                      keep_idx_out=None, n_keep_out=None):
    B, H, N, d = K.shape
    Ncap = K_out.shape[2] if K_out is not None else hidden_out.shape[1]
    Dh = hidden.shape[2] if hidden is not None else 0
    vp, vu = _vis(vis_len)
    rc = lib().vitcop_prune_step(_ptr(hidden), _ptr(K), _ptr(V), B, H, N, d, Dh, _ptr(seq_len), vis_start, vp, vu,
                                 int(Nv_cap), _ptr(label), int(budget), _ptr(hidden_out), _ptr(K_out), _ptr(V_out),
                                 Ncap, _ptr(kept_pos), _ptr(out_len), _ptr(score_out), _ptr(keep_idx_out),
                                 _ptr(n_keep_out), _ptr(workspace), workspace.numel(), _stream())
    _check(rc, "vitcop_prune_step")
    return out_len


def vitcop_prune_step_static(hidden, K, V, vis_start: int, vis_len, Nv_cap: int, budget: int, hidden_out, K_out,
                             V_out, out_len, label=None, kept_pos=None, seq_len=None, score_out=None,
                             keep_idx_out=None, n_keep_out=None):
    """``vitcop_prune_step`` on the library's built-in scratch buffer: no workspace argument, nothing allocated.

    For callers that cannot get device memory at the point of the call.  Raises ``VitcopError`` with
    ``ERR_UNSUPPORTED`` when the problem needs more than the built-in 4 MiB.  Calls share that buffer, so
    calls that could overlap on the GPU must be ordered by the caller.
    """
    B, H, N, d = K.shape
    Ncap = K_out.shape[2] if K_out is not None else hidden_out.shape[1]
    Dh = hidden.shape[2] if hidden is not None else 0
    vp, vu = _vis(vis_len)
    rc = lib().vitcop_prune_step_static(_ptr(hidden), _ptr(K), _ptr(V), B, H, N, d, Dh, _ptr(seq_len), vis_start, vp,
                                        vu, int(Nv_cap), _ptr(label), int(budget), _ptr(hidden_out), _ptr(K_out),
                                        _ptr(V_out), Ncap, _ptr(kept_pos), _ptr(out_len), _ptr(score_out),
                                        _ptr(keep_idx_out), _ptr(n_keep_out), _stream())
    _check(rc, "vitcop_prune_step_static")
    return out_len


def vitcop_collaborative_step(feat, pos, hidden, K, V, vis_start: int, budget: int, hidden_out, K_out, V_out, out_len,
                              label_out, n_clusters_out, workspace, metric: int = 0, d_c: float = 0.5, tau: float = 0.6,
                              alpha: float = 0.05, n_centers: int = 0, kept_pos=None, score_out=None, keep_idx_out=None,
                              n_keep_out=None, rho=None, delta2=None, parent=None):
    """Stage II in one call: redundancy filter + fused pruning step in quota mode, K-norm beside the clustering."""
    B, Nv, D = feat.shape
    _, H, N, d = K.shape
    Ncap = K_out.shape[2] if K_out is not None else hidden_out.shape[1]
    Dh = hidden.shape[2] if hidden is not None else 0
    p = FilterParams(int(metric), float(d_c), float(tau), float(alpha), int(n_centers))
    rc = lib().vitcop_collaborative_step(_ptr(feat), _ptr(pos), D, C.byref(p), _ptr(hidden), _ptr(K), _ptr(V), B, H, N,
                                         d, Dh, vis_start, Nv, int(budget), _ptr(hidden_out), _ptr(K_out), _ptr(V_out),
                                         Ncap, _ptr(kept_pos), _ptr(out_len), _ptr(label_out), _ptr(n_clusters_out),
                                         _ptr(rho), _ptr(delta2), _ptr(parent), _ptr(score_out), _ptr(keep_idx_out), _ptr(n_keep_out), _ptr(workspace),
                                         workspace.numel(), _stream())
    _check(rc, "vitcop_collaborative_step")
    return out_len


def vitcop_merge_clusters(hidden, vis_start: int, vis_len, label, keep_mask, merged_label, merged_count, n_merged,
                          workspace, merged=None, merged_f32=None):
    """Eq. 6: one averaged row per cluster that has non-elite tokens (``keep_mask`` 0), ascending label order."""
    B, N, Dh = hidden.shape
    Nv_cap = label.shape[1]
    Mcap = merged_label.shape[1]
    vp, vu = _vis(vis_len)
    rc = lib().vitcop_merge_clusters(_ptr(hidden), B, N, Dh, vis_start, vp, vu, Nv_cap, _ptr(label), _ptr(keep_mask),
                                     _ptr(merged), _ptr(merged_f32), _ptr(merged_label), _ptr(merged_count),
                                     _ptr(n_merged), Mcap, _ptr(workspace), workspace.numel(), _stream())
    _check(rc, "vitcop_merge_clusters")
    return n_merged


def vitcop_cls_saliency(q_cls, K, scale: float, saliency, workspace, cls_self=None):
    """Eq. 1: q_cls bf16 [B,H,d], K bf16 [B,H,M,d] (key 0 = [CLS]) -> saliency fp32 [B, M-1]."""
    B, H, M, d = K.shape
    rc = lib().vitcop_cls_saliency(_ptr(q_cls), _ptr(K), B, H, M, d, float(scale), _ptr(saliency), _ptr(cls_self),
                                   _ptr(workspace), workspace.numel(), _stream())
    _check(rc, "vitcop_cls_saliency")
    return saliency


def vitcop_kproj_knorm(hidden, W_k, H: int, d: int, K_out, workspace, vis_start: int = 0, score=None, rope_cos=None,
                       rope_sin=None, position_ids=None):
    """K = W_k x per head (+ rotary embedding) in bf16 [B,H,N,d] and Eq. 4 of the visual span from the same pass."""
    B, N, Dh = hidden.shape
    assert W_k.shape == (H * d, Dh) and K_out.shape == (B, H, N, d)
    Nv = 0 if score is None else score.shape[1]
    n_pos = 0 if rope_cos is None else rope_cos.shape[0]
    rc = lib().vitcop_kproj_knorm(_ptr(hidden), _ptr(W_k), B, N, Dh, H, d, _ptr(rope_cos), _ptr(rope_sin),
                                  _ptr(position_ids), n_pos, _ptr(K_out), int(vis_start), Nv, _ptr(score),
                                  _ptr(workspace), workspace.numel(), _stream())
    _check(rc, "vitcop_kproj_knorm")
    return K_out


def vitcop_stage_count(m: int, pi: float) -> int:
    return int(lib().vitcop_stage_count(int(m), float(pi)))


def vitcop_flops_layer(N: float, d: float) -> float:
    return float(lib().vitcop_flops_layer(float(N), float(d)))


def vitcop_visual_tokens_at_layer(l: int, m: float, pi1: float, pi2: float, pi3: float, l_s: int = 2,
                                  l_d: int = 22) -> float:
    return float(lib().vitcop_visual_tokens_at_layer(int(l), float(m), float(pi1), float(pi2), float(pi3), l_s, l_d))


def vitcop_flops_total(m: float, n_text: float, d: float, pi1: float, pi2: float, pi3: float, l_s: int = 2,
                       l_d: int = 22, n_layers: int = 32) -> float:
    return float(lib().vitcop_flops_total(float(m), float(n_text), float(d), float(pi1), float(pi2), float(pi3), l_s,
                                          l_d, n_layers))


def vitcop_cr_int(pi1: float, pi2: float, pi3: float, l_s: int = 2, l_d: int = 22, n_layers: int = 32) -> float:
    return float(lib().vitcop_cr_int(float(pi1), float(pi2), float(pi3), l_s, l_d, n_layers))


def vitcop_redundancy_filter(feat: torch.Tensor, pos: Optional[torch.Tensor], label: torch.Tensor,
                             n_clusters: torch.Tensor, workspace: torch.Tensor, metric: int = 0, d_c: float = 0.5,
                             tau: float = 0.6, alpha: float = 0.05, n_centers: int = 0, rho=None, delta2=None,
                             parent=None):
    assert feat.dtype == torch.bfloat16 and feat.dim() == 3 and label.dtype == torch.int32
    B, n, D = feat.shape
    p = FilterParams(int(metric), float(d_c), float(tau), float(alpha), int(n_centers))
    rc = lib().vitcop_redundancy_filter(_ptr(feat), _ptr(pos), B, n, D, C.byref(p), _ptr(label), _ptr(n_clusters),
                                        _ptr(rho), _ptr(delta2), _ptr(parent), _ptr(workspace), workspace.numel(),
                                        _stream())
    _check(rc, "vitcop_redundancy_filter")
    return label


def vitcop_similarity_rows(feat: torch.Tensor, metric: int, row_begin: int, row_end: int, out: torch.Tensor,
                           workspace: torch.Tensor):
    B, n, D = feat.shape
    rc = lib().vitcop_similarity_rows(_ptr(feat), B, n, D, int(metric), int(row_begin), int(row_end), _ptr(out),
                                      _ptr(workspace), workspace.numel(), _stream())
    _check(rc, "vitcop_similarity_rows")
    return out


def vitcop_set_wait_limit(limit_ns: int = 0, expire_roles: int = 0) -> None:
    """Limit of the kernels' bounded waits (0 = default 2 s); ``expire_roles`` makes the named roles give up at once."""
    _check(lib().vitcop_set_wait_limit(int(limit_ns), int(expire_roles)), "vitcop_set_wait_limit")


def vitcop_kernel_timing_begin() -> None:
    _check(lib().vitcop_kernel_timing_begin(), "vitcop_kernel_timing_begin")


def vitcop_kernel_timing_end(capacity: int = 32) -> dict:
    """{kernel name: (launches, total milliseconds)} of the kernels launched since ``vitcop_kernel_timing_begin``."""
    buf = (KernelTime * capacity)()
    n = C.c_int(0)
    _check(lib().vitcop_kernel_timing_end(buf, capacity, C.byref(n)), "vitcop_kernel_timing_end")
    return {buf[i].name.decode(): (int(buf[i].launches), float(buf[i].total_ms)) for i in range(n.value)}


# ----------------------------------------------------------------------------------------------
def bf16_tensor(bits, device="cuda") -> torch.Tensor:
    """uint16 numpy bit patterns -> bf16 torch tensor on ``device`` (no rounding involved)."""
    import numpy as np
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16))
    return t.to(device).view(torch.bfloat16)


def bf16_bits(t: torch.Tensor):
    """bf16 torch tensor -> uint16 numpy bit patterns."""
    import numpy as np
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
