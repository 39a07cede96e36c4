"""ctypes wrappers around ``vitcop_oracle.cpp`` (test infrastructure; see the package docstring)."""
from __future__ import annotations

import ctypes as C
import hashlib
import os
import platform
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "vitcop_oracle.cpp")
_lib = None


def _host_tag() -> str:
    flags = ""
    try:
        with open("/proc/cpuinfo") as fh:
            for line in fh:
                if line.startswith("flags"):
                    flags = line
                    break
    except OSError:
        pass
    with open(_SRC, "rb") as fh:
        src = fh.read()
    return hashlib.sha1(src + flags.encode() + platform.machine().encode()).hexdigest()[:12]


def build(verbose: bool = False) -> str:
    """Compile the oracle for this host (no-op when an up-to-date object exists); returns its path."""
    out = os.path.join(_HERE, f"_oracle_{_host_tag()}.so")
    if not os.path.exists(out):
        tmp = out + f".tmp{os.getpid()}"
        cmd = ["g++", "-O3", "-march=native", "-std=c++17", "-fopenmp", "-shared", "-fPIC", _SRC, "-o", tmp]
        if verbose:
            print(" ".join(cmd))
        subprocess.check_call(cmd)
        os.replace(tmp, out)
    return out


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_cr_int.restype = C.c_double
        _lib.oracle_flops_layer.restype = C.c_double
        _lib.oracle_visual_tokens_at_layer.restype = C.c_double
        _lib.oracle_flops_vitcop.restype = C.c_double
    return _lib


def num_threads() -> int:
    """Threads the OpenMP loops of the oracle will use."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env)
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _u16(a: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


# ------------------------------------------------------------------------------------------ O1
def knorm(K_bits: np.ndarray, vis_start: int, vis_len) -> np.ndarray:
    """Eq. 4 on bf16 bits K [B,H,N,d] -> float64 [B, max vis_len] (NaN-free; unused tail is 0)."""
    K_bits = _u16(K_bits)
    B, H, N, d = K_bits.shape
    if np.isscalar(vis_len):
        vl, uni, cap = None, int(vis_len), int(vis_len)
    else:
        vl = np.ascontiguousarray(vis_len, dtype=np.int32)
        uni, cap = 0, int(vl.max()) if vl.size else 0
    out = np.zeros((B, max(cap, 0)), dtype=np.float64)
    lib().oracle_knorm(_p(K_bits), B, H, N, d, C.c_int64(H * N * d), C.c_int64(N * d), C.c_int64(d),
                       vis_start, _p(vl), uni, _p(out), max(cap, 0))
    return out


# ------------------------------------------------------------------------------------------ O2 / O4
def select_plain(score: np.ndarray, budget: int, largest: bool = False) -> np.ndarray:
    """Plain top-k of one sequence; returns ascending int32 indices."""
    s = np.ascontiguousarray(score, dtype=np.float64)
    n = s.shape[0]
    keep = np.empty(max(n, 1), dtype=np.int32)
    k = lib().oracle_select_plain(_p(s), n, int(budget), int(bool(largest)), _p(keep))
    return keep[:k].copy()


def select_quota(score: np.ndarray, label: np.ndarray, budget: int):
    """Eq. 5 / Algorithm 3 elites of one sequence.

    Returns (keep_idx ascending or None when budget < N_c, N_c, quota[n] indexed by label value).
    """
    s = np.ascontiguousarray(score, dtype=np.float64)
    lab = np.ascontiguousarray(label, dtype=np.int32)
    n = s.shape[0]
    keep = np.empty(max(n, 1), dtype=np.int32)
    nc = C.c_int32(0)
    quota = np.zeros(max(n, 1), dtype=np.int32)
    k = lib().oracle_select_quota(_p(s), _p(lab), n, int(budget), _p(keep), C.byref(nc), _p(quota))
    return (None if k < 0 else keep[:k].copy()), int(nc.value), quota[:n]


# ------------------------------------------------------------------------------------------ O3
def feature_distance(feat_bits: np.ndarray, metric: int = 0, rows: Optional[Tuple[int, int]] = None,
                     want_d2: bool = True, want_sim: bool = True):
    """Pairwise squared feature distance and similarity of one sample, bf16 bits [n, D].

    Returns (d2, sim), each float64 [rows, n] (or None when not wanted).
    """
    f = _u16(feat_bits)
    n, D = f.shape
    r0, r1 = (0, n) if rows is None else rows
    d2 = np.empty((r1 - r0, n), dtype=np.float64) if want_d2 else None
    sim = np.empty((r1 - r0, n), dtype=np.float64) if want_sim else None
    lib().oracle_feature_distance_rows(_p(f), n, D, int(metric), r0, r1, _p(d2), _p(sim))
    return d2, sim


def vic_density(d2: np.ndarray, d_c: float) -> np.ndarray:
    d2 = np.ascontiguousarray(d2, dtype=np.float64)
    n = d2.shape[0]
    rho = np.empty(n, dtype=np.float64)
    lib().oracle_vic_density(_p(d2), n, C.c_double(d_c), _p(rho))
    return rho


def vic_parents(d2: np.ndarray, pos: Optional[np.ndarray], rho: np.ndarray, tau: float,
                tol_rho: float = 0.0, tol_d2_abs: float = 0.0, tol_d2_rel: float = 0.0, tol_sp: float = 0.0,
                want_fragile: bool = False):
    """Eq. 3 -> (delta2 [n] float64 with +inf for orphans, parent [n] int32, fragile [n] uint8 or None)."""
    d2 = np.ascontiguousarray(d2, dtype=np.float64)
    n = d2.shape[0]
    rho = np.ascontiguousarray(rho, dtype=np.float64)
    p = None if pos is None else np.ascontiguousarray(pos, dtype=np.float32)
    delta2 = np.empty(n, dtype=np.float64)
    parent = np.empty(n, dtype=np.int32)
    frag = np.zeros(n, dtype=np.uint8) if want_fragile else None
    lib().oracle_vic_parents(_p(d2), _p(p), _p(rho), n, C.c_double(tau), _p(delta2), _p(parent), _p(frag),
                             C.c_double(tol_rho), C.c_double(tol_d2_abs), C.c_double(tol_d2_rel), C.c_double(tol_sp))
    return delta2, parent, frag


def vic_centers(rho: np.ndarray, delta2: np.ndarray, n_centers: int):
    """Algorithm 2 step 3 -> (is_center [n] uint8, gamma [n] float64, rank order [n] int32)."""
    rho = np.ascontiguousarray(rho, dtype=np.float64)
    delta2 = np.ascontiguousarray(delta2, dtype=np.float64)
    n = rho.shape[0]
    isc = np.zeros(n, dtype=np.uint8)
    gamma = np.empty(n, dtype=np.float64)
    rank = np.empty(n, dtype=np.int32)
    lib().oracle_vic_centers(_p(rho), _p(delta2), n, int(n_centers), _p(isc), _p(gamma), _p(rank))
    return isc, gamma, rank


def vic_num_centers(n: int, alpha: float) -> int:
    return int(lib().oracle_vic_num_centers(int(n), C.c_double(alpha)))


def vic_labels(d2: np.ndarray, rho: np.ndarray, parent: np.ndarray, is_center: np.ndarray) -> np.ndarray:
    d2 = np.ascontiguousarray(d2, dtype=np.float64)
    rho = np.ascontiguousarray(rho, dtype=np.float64)
    parent = np.ascontiguousarray(parent, dtype=np.int32)
    isc = np.ascontiguousarray(is_center, dtype=np.uint8)
    n = rho.shape[0]
    label = np.empty(n, dtype=np.int32)
    lib().oracle_vic_labels(_p(d2), _p(rho), _p(parent), _p(isc), n, _p(label))
    return label


def vic(feat_bits: np.ndarray, pos: Optional[np.ndarray], metric: int, d_c: float, tau: float, n_centers: int,
        tols: Optional[dict] = None) -> dict:
    """Algorithm 2 on one sample (bf16 bits [n, D], fp32 positions [n, 2] or None)."""
    d2, sim = feature_distance(feat_bits, metric)
    rho = vic_density(d2, d_c)
    t = tols or {}
    delta2, parent, frag = vic_parents(d2, pos, rho, tau, want_fragile=tols is not None, **t)
    isc, gamma, rank = vic_centers(rho, delta2, n_centers)
    label = vic_labels(d2, rho, parent, isc)
    return dict(d2=d2, sim=sim, rho=rho, delta2=delta2, parent=parent, fragile=frag, is_center=isc,
                gamma=gamma, rank=rank, label=label, n_clusters=int(isc.sum()))


# ------------------------------------------------------------------------------------------ O5
def compact(hidden: Optional[np.ndarray], K: Optional[np.ndarray], V: Optional[np.ndarray], seq_len: int,
            vis_start: int, vis_len: int, keep_idx: np.ndarray, Ncap: int):
    """Compaction of one sample: hidden [N,Dh], K/V [H,N,d] bf16 bits -> dict of outputs."""
    keep_idx = np.ascontiguousarray(keep_idx, dtype=np.int32)
    ref = K if K is not None else V
    if ref is not None:
        H, N, d = ref.shape
    else:
        H, N, d = 0, hidden.shape[0], 0
    Dh = hidden.shape[1] if hidden is not None else 0
    ho = np.zeros((Ncap, Dh), dtype=np.uint16) if hidden is not None else None
    Ko = np.zeros((H, Ncap, d), dtype=np.uint16) if K is not None else None
    Vo = np.zeros((H, Ncap, d), dtype=np.uint16) if V is not None else None
    pos = np.full(Ncap, -1, dtype=np.int32)
    out_len = lib().oracle_compact(_p(None if hidden is None else _u16(hidden)), _p(None if K is None else _u16(K)),
                                   _p(None if V is None else _u16(V)), H, N, d, Dh, int(seq_len), int(vis_start),
                                   int(vis_len), _p(keep_idx), int(keep_idx.shape[0]), _p(ho), _p(Ko), _p(Vo),
                                   int(Ncap), _p(pos))
    return dict(hidden=ho, K=Ko, V=Vo, kept_pos=pos, out_len=int(out_len))


# ------------------------------------------------------------------------------------------ schedule
def stage_count(m: int, pi: float) -> int:
    return int(lib().oracle_stage_count(int(m), C.c_double(pi)))


def cr_int(pi1: float, pi2: float, pi3: float, l_s: int = 2, l_d: int = 22, n_layers: int = 32) -> float:
    return float(lib().oracle_cr_int(C.c_double(pi1), C.c_double(pi2), C.c_double(pi3), l_s, l_d, n_layers))


# ------------------------------------------------------------------------------------------ O7 / O8 / cost model
def merge_clusters(hidden: np.ndarray, vis_start: int, label: np.ndarray, keep_mask: np.ndarray):
    """Eq. 6 on one sample: hidden bf16 bits [N, Dh], label / keep_mask [n].

    Returns (merged float64 [M, Dh], merged_label int32 [M], merged_count int32 [M]), clusters in ascending label."""
    h = _u16(hidden)
    N, Dh = h.shape
    lab = np.ascontiguousarray(label, dtype=np.int32)
    keep = np.ascontiguousarray(keep_mask, dtype=np.uint8)
    n = lab.shape[0]
    cap = max(n, 1)
    merged = np.zeros((cap, Dh), dtype=np.float64)
    mlab = np.zeros(cap, dtype=np.int32)
    mcnt = np.zeros(cap, dtype=np.int32)
    m = lib().oracle_merge_clusters(_p(h), N, Dh, int(vis_start), n, _p(lab), _p(keep), _p(merged), _p(mlab), _p(mcnt),
                                    cap)
    return merged[:m].copy(), mlab[:m].copy(), mcnt[:m].copy()


def cls_saliency(q_bits: np.ndarray, K_bits: np.ndarray, scale: float):
    """Eq. 1 on one image: q bf16 bits [H, d], K [H, M, d] (key 0 = [CLS]) -> (S float64 [M-1], self-attention of [CLS])."""
    q, K = _u16(q_bits), _u16(K_bits)
    H, M, d = K.shape
    S = np.zeros(max(M - 1, 0), dtype=np.float64)
    c = C.c_double(0.0)
    lib().oracle_cls_saliency(_p(q), _p(K), H, M, d, C.c_double(scale), _p(S), C.byref(c))
    return S, float(c.value)


def kproj_knorm(hidden_bits: np.ndarray, W_bits: np.ndarray, H: int, d: int, cos: Optional[np.ndarray] = None,
                sin: Optional[np.ndarray] = None, position: Optional[np.ndarray] = None):
    """K = W_k t per head (+ rotary embedding), rounded to bf16, and its Eq. 4 norm, for one sample.

    hidden bf16 bits [N, Dh], W bf16 bits [H*d, Dh], cos / sin float64 [n_pos, d/2] or None, position int32 [N] or None.
    Returns (K float64 [H, N, d] before rounding, K bf16 bits [H, N, d], score float64 [N])."""
    h, W = _u16(hidden_bits), _u16(W_bits)
    N, Dh = h.shape
    assert W.shape == (H * d, Dh)
    c = None if cos is None else np.ascontiguousarray(cos, dtype=np.float64)
    s = None if sin is None else np.ascontiguousarray(sin, dtype=np.float64)
    pos = None if position is None else np.ascontiguousarray(position, dtype=np.int32)
    K64 = np.empty((H, N, d), dtype=np.float64)
    Kb = np.empty((H, N, d), dtype=np.uint16)
    score = np.empty(N, dtype=np.float64)
    lib().oracle_kproj_knorm(_p(h), _p(W), N, Dh, H, d, _p(c), _p(s), _p(pos), _p(K64), _p(Kb), _p(score))
    return K64, Kb, score


def flops_layer(N: float, d: float) -> float:
    return float(lib().oracle_flops_layer(C.c_double(N), C.c_double(d)))


def visual_tokens_at_layer(l: int, m: float, pi1: float, pi2: float, pi3: float, l_s: int = 2, l_d: int = 22) -> float:
    return float(lib().oracle_visual_tokens_at_layer(int(l), C.c_double(m), C.c_double(pi1), C.c_double(pi2),
                                                     C.c_double(pi3), l_s, l_d))


def flops_vitcop(m: float, n_text: float, d: float, pi1: float, pi2: float, pi3: float, l_s: int = 2, l_d: int = 22,
                 n_layers: int = 32) -> float:
    return float(lib().oracle_flops_vitcop(C.c_double(m), C.c_double(n_text), C.c_double(d), C.c_double(pi1),
                                           C.c_double(pi2), C.c_double(pi3), l_s, l_d, n_layers))


__all__ = [n for n in dir() if not n.startswith("_") and n not in ("C", "np", "os", "hashlib", "platform",
                                                                   "subprocess", "Optional", "Tuple", "annotations")]
