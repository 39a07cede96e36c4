"""Seeded synthetic inputs for the ViTCoP pruning operator chain.

This module only *generates inputs* (random tensors shaped like LLaVA-1.5,
LLaVA-NeXT AnyRes and video-LLM prefill workloads).  It contains none of the
method's arithmetic and is the one module shared by the CUDA path's tests,
the CPU oracle's tests and the benchmark.  It depends on numpy alone.

All bf16 tensors are returned as ``uint16`` numpy arrays holding the bf16 bit
pattern (round-to-nearest-even from fp32), so that the CPU oracle and the GPU
kernels consume exactly the same bits.

Every "N(0, s)" / "log-normal(0, s)" below takes ``s`` as a standard
deviation.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np

__all__ = [
    "Workload", "WORKLOADS", "workload", "f32_to_bf16_bits", "bf16_bits_to_f32",
    "make_features", "make_positions", "make_kv", "make_hidden", "make_scores", "make_labels", "make_cls_qk",
]


# --------------------------------------------------------------------------- bf16 helpers
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 -> bf16 (round-to-nearest-even); returns the uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    out = (r >> np.uint32(16)).astype(np.uint16)
    nan = np.isnan(x)
    if nan.any():
        out[nan] = np.uint16(0x7FC0)
    return out


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp32."""
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(seed: int, cfg: int, tensor_id: int, step: int = 0) -> np.random.Generator:
    """Counter-based generator keyed by (seed, config, tensor id, step)."""
    key = (np.uint64(seed) << np.uint64(32)) ^ (np.uint64(cfg) << np.uint64(20)) \
        ^ (np.uint64(tensor_id) << np.uint64(8)) ^ np.uint64(step)
    return np.random.Generator(np.random.Philox(key=int(key)))


# --------------------------------------------------------------------------- workload table
@dataclass(frozen=True)
class Workload:
    """Shapes and distributions of one synthetic workload."""
    name: str
    cfg: int                 # index, also folded into the generator key
    B: int                   # batch
    H: int                   # KV heads
    d: int                   # head dim
    Nv: int                  # visual tokens entering step 0
    T: int                   # text tokens (a prefix: vis_start == T)
    D: int                   # vision feature dim
    Dh: int                  # LLM hidden size
    budgets: Tuple[int, ...]  # keep budget of each successive pruning step
    n_centers: int           # VIC cluster centres (integer form of ceil(n*alpha), alpha = 0.05)
    layout: str              # "image24" | "anyres" | "video" | "image128"
    dup_rate: float = 0.0    # fraction of near-duplicate tokens
    dup_sigma: float = 0.01
    drift_sigma: float = 0.05
    outlier_rate: float = 0.0
    outlier_scale: float = 10.0
    k_sigma: float = 0.5     # std of the log of the per-token K scale
    d_c: float = 0.5         # VIC cutoff distance used with the cosine metric
    tau: float = 0.6         # VIC spatial threshold on [0,1]^2 coordinates
    seed: int = 0

    @property
    def vis_start(self) -> int:
        return self.T

    @property
    def N(self) -> int:
        return self.T + self.Nv


WORKLOADS: Dict[str, Workload] = {
    # LLaVA-1.5-7B-shaped single image
    "c0": Workload("c0", 0, 1, 32, 128, 576, 64, 1024, 4096, (192, 128, 64), 29, "image24", dup_rate=0.2),
    # LLaVA-1.5-7B-shaped batch 16, extreme pruning
    "c1": Workload("c1", 1, 16, 32, 128, 576, 64, 1024, 4096, (64,), 29, "image24", dup_rate=0.2),
    # LLaVA-NeXT AnyRes-shaped batch 8
    "c2": Workload("c2", 2, 8, 32, 128, 2880, 64, 1024, 4096, (640, 320, 160), 144, "anyres", dup_rate=0.3),
    # video-LLM-shaped batch 4 (32 frames x 144 tokens)
    "c3": Workload("c3", 3, 4, 32, 128, 4608, 64, 1024, 4096, (1152, 576, 288), 231, "video"),
    # long-video GQA stress, batch 2
    "c4": Workload("c4", 4, 2, 4, 128, 16384, 128, 1280, 3584, (2048, 1024, 512), 820, "image128",
                   dup_rate=0.4, outlier_rate=0.01),
    # tiny case for smoke tests: several tiles plus a ragged tail
    "tiny": Workload("tiny", 9, 2, 4, 64, 200, 9, 128, 256, (96, 40, 7), 10, "image24", dup_rate=0.2),
}


def workload(name: str) -> Workload:
    return WORKLOADS[name]


# --------------------------------------------------------------------------- positions
def _grid_positions(rows: int, cols: int) -> np.ndarray:
    r, c = np.meshgrid(np.arange(rows), np.arange(cols), indexing="ij")
    p = np.stack([(c + 0.5) / cols, (r + 0.5) / rows], axis=-1).reshape(-1, 2)
    return p.astype(np.float32)


def make_positions(w: Workload, n: Optional[int] = None) -> np.ndarray:
    """fp32 [B, n, 2] token coordinates normalised to the unit square (x, y)."""
    n = w.Nv if n is None else n
    if w.layout == "image24":
        side = 24
        base = _grid_positions(side, side)
        reps = -(-n // base.shape[0])
        p = np.tile(base, (reps, 1))[:n]
    elif w.layout == "image128":
        p = _grid_positions(128, 128)[:n]
    elif w.layout == "anyres":
        base = _grid_positions(24, 24)                        # overview tile covers the whole image
        tiles = [base]
        for ty in range(2):
            for tx in range(2):
                r, c = np.meshgrid(np.arange(24), np.arange(24), indexing="ij")
                q = np.stack([(24 * tx + c + 0.5) / 48.0, (24 * ty + r + 0.5) / 48.0], axis=-1)
                tiles.append(q.reshape(-1, 2).astype(np.float32))
        p = np.concatenate(tiles, 0)[:n]
    elif w.layout == "video":
        frame = _grid_positions(12, 12)
        reps = -(-n // 144)
        p = np.tile(frame, (reps, 1))[:n]                      # time is ignored
    else:
        raise ValueError(w.layout)
    return np.ascontiguousarray(np.broadcast_to(p[None], (w.B, n, 2)), dtype=np.float32)


# --------------------------------------------------------------------------- vision features
def _near_dups_grid(rng, f: np.ndarray, side_r: int, side_c: int, n_dup: int, sigma: float) -> np.ndarray:
    """Replace ``n_dup`` seeded tokens by (a non-replaced token within 4 grid cells) + noise."""
    n = f.shape[0]
    order = rng.permutation(n)
    replaced = np.zeros(n, dtype=bool)
    replaced[order[:n_dup]] = True
    rr, cc = np.divmod(np.arange(n), side_c)
    rr = rr % side_r
    for i in order[:n_dup]:
        src = -1
        for _ in range(64):
            dr, dc = rng.integers(-4, 5, size=2)
            r2, c2 = rr[i] + dr, cc[i] + dc
            if (dr == 0 and dc == 0) or not (0 <= r2 < side_r and 0 <= c2 < side_c):
                continue
            j = (i // (side_r * side_c)) * side_r * side_c + r2 * side_c + c2
            if j < n and not replaced[j]:
                src = j
                break
        if src < 0:                                            # crowded neighbourhood: any clean token
            src = int(np.flatnonzero(~replaced)[0])
        f[i] = f[src] + sigma * rng.standard_normal(f.shape[1], dtype=np.float32)
    return f


def make_features(w: Workload, n: Optional[int] = None, B: Optional[int] = None) -> np.ndarray:
    """bf16 bits [B, n, D]: vision features with the workload's redundancy structure."""
    n = w.Nv if n is None else n
    B = w.B if B is None else B
    out = np.empty((B, n, w.D), dtype=np.uint16)
    for b in range(B):
        rng = _rng(w.seed, w.cfg, 1, b)
        if w.layout == "video":
            per = 144
            frames = -(-n // per)
            cur = rng.standard_normal((per, w.D), dtype=np.float32)
            cur = bf16_bits_to_f32(f32_to_bf16_bits(cur))
            fs = [cur]
            for _ in range(1, frames):
                cur = cur + np.float32(w.drift_sigma) * rng.standard_normal((per, w.D), dtype=np.float32)
                cur = bf16_bits_to_f32(f32_to_bf16_bits(cur))  # each frame is rounded before the next drifts
                fs.append(cur)
            f = np.concatenate(fs, 0)[:n]
        else:
            f = rng.standard_normal((n, w.D), dtype=np.float32)
            n_dup = int(np.floor(w.dup_rate * n))
            if w.layout == "anyres" and n_dup > 0 and n >= 5 * 576:
                # crop tokens copy the overview-tile token that covers the same image location;
                # crop rows/columns that touch an inner tile boundary are taken first.
                crop = np.arange(576, 5 * 576)
                t = (crop - 576) // 576
                ty, tx = t // 2, t % 2
                r, c = np.divmod((crop - 576) % 576, 24)
                inner = ((tx == 0) & (c == 23)) | ((tx == 1) & (c == 0)) | ((ty == 0) & (r == 23)) | ((ty == 1) & (r == 0))
                first = crop[inner]
                rest = rng.permutation(crop[~inner])
                chosen = np.concatenate([first, rest])[:n_dup]
                t = (chosen - 576) // 576
                ty, tx = t // 2, t % 2
                r, c = np.divmod((chosen - 576) % 576, 24)
                src = ((24 * ty + r) // 2) * 24 + (24 * tx + c) // 2
                f[chosen] = f[src] + np.float32(w.dup_sigma) * rng.standard_normal((chosen.size, w.D), dtype=np.float32)
            elif n_dup > 0:
                side = 128 if w.layout == "image128" else 24
                f = _near_dups_grid(rng, f, side, side, n_dup, np.float32(w.dup_sigma))
            if w.outlier_rate > 0:
                n_out = int(np.floor(w.outlier_rate * n))
                idx = rng.permutation(n)[:n_out]
                f[idx] *= np.float32(w.outlier_scale)
        out[b] = f32_to_bf16_bits(f)
    return out


# --------------------------------------------------------------------------- LLM-side tensors
def make_kv(w: Workload, step: int, n_vis: int, B: Optional[int] = None) -> Tuple[np.ndarray, np.ndarray]:
    """bf16 bits K, V of shape [B, H, T + n_vis, d] for pruning step ``step``.

    K = N(0,1) * exp(N(0, k_sigma)) with one scale per token (text tokens included),
    V = N(0,1).  A later step stands for a later layer, hence a fresh tensor.
    """
    B = w.B if B is None else B
    N = w.T + n_vis
    K = np.empty((B, w.H, N, w.d), dtype=np.uint16)
    V = np.empty((B, w.H, N, w.d), dtype=np.uint16)
    for b in range(B):
        rng = _rng(w.seed, w.cfg, 2 + 2 * step, b)
        scale = np.exp(np.float32(w.k_sigma) * rng.standard_normal(N, dtype=np.float32)).astype(np.float32)
        k = rng.standard_normal((w.H, N, w.d), dtype=np.float32) * scale[None, :, None]
        K[b] = f32_to_bf16_bits(k)
        rng2 = _rng(w.seed, w.cfg, 3 + 2 * step, b)
        V[b] = f32_to_bf16_bits(rng2.standard_normal((w.H, N, w.d), dtype=np.float32))
    return K, V


def make_hidden(w: Workload, B: Optional[int] = None) -> np.ndarray:
    """bf16 bits [B, N, Dh] residual-stream rows, N(0,1)."""
    B = w.B if B is None else B
    out = np.empty((B, w.N, w.Dh), dtype=np.uint16)
    for b in range(B):
        rng = _rng(w.seed, w.cfg, 40, b)
        out[b] = f32_to_bf16_bits(rng.standard_normal((w.N, w.Dh), dtype=np.float32))
    return out


def make_scores(seed: int, B: int, n: int, kind: str = "lognormal") -> np.ndarray:
    """fp32 [B, n] stand-alone score arrays for selection tests."""
    rng = _rng(seed, 31, 7, n)
    if kind == "lognormal":
        return np.exp(0.5 * rng.standard_normal((B, n))).astype(np.float32)
    if kind == "ties":                                          # few distinct values: ties everywhere
        return rng.integers(0, 4, size=(B, n)).astype(np.float32)
    if kind == "equal":
        return np.full((B, n), 1.25, dtype=np.float32)
    if kind == "signed":
        return rng.standard_normal((B, n)).astype(np.float32)
    raise ValueError(kind)


def make_labels(seed: int, B: int, n: int, n_clusters: int, skew: float = 0.0) -> np.ndarray:
    """int32 [B, n] random cluster labels; a label is the token index of its cluster's centre.

    Cluster sizes are multinomial-even by default; ``skew`` in (0, 1) first hands that share of the tokens to one
    cluster (a large background cluster beside many small ones)."""
    rng = _rng(seed, 32, 8, n)
    out = np.empty((B, n), dtype=np.int32)
    for b in range(B):
        centres = np.sort(rng.permutation(n)[:n_clusters]).astype(np.int32)
        lab = centres[rng.integers(0, n_clusters, size=n)]
        if skew > 0.0:
            big = centres[int(rng.integers(0, n_clusters))]
            lab[rng.random(n) < skew] = big
        lab[centres] = centres                                  # a centre carries its own index
        out[b] = lab
    return out


def make_cls_qk(seed: int, B: int, H: int, M: int, d: int, salient: float = 0.05) -> Tuple[np.ndarray, np.ndarray]:
    """bf16 bits q [B, H, d] and K [B, H, M, d] of one vision-encoder layer (key 0 belongs to [CLS]).

    Keys are N(0,1); a fraction ``salient`` of the tokens gets a component along the head's query, so that the
    [CLS] attention row is peaked on a few tokens the way a trained encoder's is (shapes of CLIP ViT-L/14-336:
    H = 16, d = 64, M = 577)."""
    rng = _rng(seed, 33, 9, M)
    q = rng.standard_normal((B, H, d), dtype=np.float32)
    K = rng.standard_normal((B, H, M, d), dtype=np.float32)
    n_sal = max(1, int(salient * M))
    for b in range(B):
        idx = rng.permutation(M)[:n_sal]
        gain = rng.uniform(0.5, 1.5, size=n_sal).astype(np.float32)
        K[b, :, idx] += (gain[:, None, None] * q[b][None, :, :]).astype(np.float32)
    return f32_to_bf16_bits(q), f32_to_bf16_bits(K)
