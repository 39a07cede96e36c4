// Interface between the tensor-core Gram sweep (gram.cu) and the rest of the redundancy filter (filter.cu).
#pragma once

#include "internal.cuh"

namespace vitcop {

constexpr int kGramBM = 128;   // rows of an output tile (UMMA M)

// GRAM_DIAG visits only the diagonal tiles and turns g_ii into the per-token factors w and a.
enum GramMode { GRAM_RHO = 0, GRAM_DELTA = 1, GRAM_SIM = 2, GRAM_DIAG = 3 };

// Tiling of the symmetric sweeps (GRAM_RHO, GRAM_DELTA).  Only tiles that hold a pair (i, j) with i < j are
// visited; a pair contributes to its row token i ("row side") and to its column token j ("column side").
// Tiles are numbered column-tile major inside one sample: column tile tj holds the row tiles
// 0 .. min(TI, R * (tj + 1)) - 1 with R = BN / kGramBM, and starts at offset R * tj * (tj + 1) / 2.
struct GramTiling {
    int BN;            // columns of an output tile: 128 or 256
    int R;             // BN / kGramBM
    int TI, TJ;        // row tiles, column tiles per sample
    int tiles_per_b;   // visited tiles per sample
    int n_pad;         // padded token count of one partial-sum slot
    __host__ __device__ int slots() const { return TJ + TI; }   // rho partial slots per sample: TJ row-side + TI column-side
};

inline GramTiling make_gram_tiling(int n, int BN) {
    GramTiling t;
    t.BN = BN;
    t.R = BN / kGramBM;
    t.TI = (n + kGramBM - 1) / kGramBM;
    t.TJ = (n + BN - 1) / BN;
    const int last = t.R * t.TJ < t.TI ? t.R * t.TJ : t.TI;
    t.tiles_per_b = t.TJ > 0 ? t.R * (t.TJ - 1) * t.TJ / 2 + last : 0;
    t.n_pad = t.TI * kGramBM;
    return t;
}

// Tile t of the symmetric numbering -> (sample, row tile, column tile).
__host__ __device__ inline void decode_sym_tile(const GramTiling& tl, long long t, int& b, int& ti, int& tj) {
    b = (int)(t / tl.tiles_per_b);
    const int r = (int)(t - (long long)b * tl.tiles_per_b);
    const int R = tl.R;
#ifdef __CUDA_ARCH__
    int q = (int)((sqrtf(8.f * (float)r / (float)R + 1.f) - 1.f) * 0.5f);
#else
    int q = 0;
#endif
    while (q > 0 && R * q * (q + 1) / 2 > r) --q;
    while (R * (q + 1) * (q + 2) / 2 <= r) ++q;
    tj = q;
    ti = r - R * q * (q + 1) / 2;
}

// The density sweep keeps the Gram values it computes: tile t (symmetric numbering, all samples) occupies
// kGramBM * BN floats at t * kGramBM * BN, stored in groups of four columns -- element (row r, column c) at
// ((c / 4) * kGramBM + r) * 4 + c % 4 -- so that the 32 lanes of a warp, one row each, write and read 512
// contiguous bytes per instruction.  The delta pass (delta_pass.cu) reads them back instead of recomputing them.
__host__ __device__ constexpr size_t gram_tile_floats(int BN) { return (size_t)kGramBM * BN; }

// Eq. 3 needs every pair a second time, once the densities are known.  A long sample's Gram values are kept by the
// density sweep and read back by the delta pass (4 bytes per pair against 2 D flop to recompute it); the pass is cheap
// because most pairs fail a bound test, and the bounds only bite when every token has thousands of candidates.  For
// shorter samples the Gram sweep is simply run again with the Eq. 3 epilogue (its loads and tensor-core work overlap
// the density sweep's tail).  Both routes give the same bits.  Measured on one B200 (step of Stage II, microseconds):
// 2 x 16384 tokens 1042 kept / 1135 recomputed; 8 x 2880 tokens 257 / 232; 4 x 4608 tokens 276 / 236.
constexpr int kKeepTilesFromTokens = 8192;
bool gram_keeps_tiles(int B, int n);

// Bounded device waits of the Gram kernels: the time after which a wait gives up (0 = the default of 2 s) and, for
// failure-handling tests, the roles whose waits give up at once (1 load warp, 2 MMA warp, 4 epilogue warps).
// Applies to launches made after the call.
void gram_set_wait_debug(unsigned long long limit_ns, int expire_roles);
unsigned long long gram_wait_limit_ns();

// Tile width the sweeps use for a problem: wide tiles halve the operand traffic per flop, narrow tiles fill
// the SMs when the problem is small.
int gram_pick_bn(int B, int n);

struct GramArgs {
    int B, n, D;
    int row0, row_end;          // GRAM_SIM: rows [row0, row_end) are produced
    int metric;                 // 0 cosine, 1 euclid
    float c2;                   // -(log2 e) / d_c^2
    float tau2;                 // tau^2; < 0: no spatial test
    const float* w;             // [B, n] factor multiplying the Gram value (cosine 1/|f|, euclid 1)
    const float* a;             // [B, n] additive term (cosine 1, euclid |f|^2):  d^2 = a_i + a_j - 2 g w_i w_j
    const float* rho;           // [B, n]                          (GRAM_DELTA)
    const float* pos;           // [B, n, 2] or nullptr            (GRAM_DELTA)
    float* part;                // [B, slots, n_pad] rho partials  (GRAM_RHO)
    unsigned long long* best;   // [B, n] packed (d2 bits << 32 | index), ~0 = none   (GRAM_DELTA)
    float* sim_out;             // [B, row_end - row0, n]          (GRAM_SIM)
    float* gram_tiles;          // Gram values of every visited tile, written by GRAM_RHO sweeps when not null
    float* w_out;               // [B, n] factors written by GRAM_DIAG (best, if given, is reset to ~0 as well)
    float* a_out;               // [B, n]
    float* rho_out;             // [B, n] written by the resident sweep (same memory as rho)
    float* rho_user;            // [B, n] optional copy of rho for the caller
    unsigned int* grid_sync;    // zeroed counter for the resident sweep's grid-wide barrier
    unsigned int* diag_ready;   // zeroed flags [B, ceil(n / 128)] of the resident sweep: factors of a row block written
    // Optional K-norm (Eq. 4) for the resident sweep's load and MMA warps to stream once their own work is issued:
    // K bf16 [kn_B, kn_H, kn_N, kn_d] dense, span [kn_vis_start, kn_vis_start + kn_Nv), score [kn_B, kn_Nv].
    // Only shapes gram_resident_takes_knorm accepts.
    const void* kn_K;
    float* kn_score;
    int kn_B, kn_H, kn_N, kn_d, kn_vis_start, kn_Nv;
    float4* bbox;               // [B, ceil(n / 128)] bounding box (min x, min y, max x, max y) of every row block's
                                // positions, or nullptr: written by GRAM_DIAG, read where whole tiles are skipped
    const int32_t* kept;        // delta pass, optional: numbers of the tiles to read, ascending; nullptr = all of them
    const int32_t* n_kept;      // their count (device)
    int* status;                // device status word
};

// Eq. 3 only pairs tokens within the spatial radius, so a tile whose row block lies farther than the radius from its
// column blocks cannot contribute: the density sweep need not keep it and the delta pass need not read it.  The
// distance between the bounding boxes is taken with the operations of the per-pair test (fp32 differences, squares
// joined by one fma), all of them monotone, so it never exceeds the distance of any pair of the tile: what is
// skipped is exactly what the per-pair test would have rejected.  `bbox_b`: the sample's boxes.
__device__ __forceinline__ bool tile_outside_radius(const float4* __restrict__ bbox_b, const GramTiling& t, int ti, int tj,
                                                    float tau2) {
    const float4 r = bbox_b[ti];
    float4 c = bbox_b[t.R * tj];
    for (int k = 1; k < t.R; ++k) {
        if (t.R * tj + k >= t.TI) break;
        const float4 o = bbox_b[t.R * tj + k];
        c = make_float4(fminf(c.x, o.x), fminf(c.y, o.y), fmaxf(c.z, o.z), fmaxf(c.w, o.w));
    }
    const float dx = fmaxf(0.f, fmaxf(r.x - c.z, c.x - r.z));
    const float dy = fmaxf(0.f, fmaxf(r.y - c.w, c.y - r.w));
    return fmaf(dx, dx, dy * dy) > tau2;
}

// rho of token i of one sample from the partial sums of the tiles that hold it, in a fixed order (reproducible
// bits): the row-side slots of the column tiles that pair row tile i / 128 with later tokens, then the column-side
// slots of the row tiles that pair column tile i / BN with earlier tokens.  `p` points at the sample's slot 0, token i.
__host__ __device__ inline float rho_from_partials(const float* p, const GramTiling& t, int i) {
    const int ti = i / kGramBM, tj = i / t.BN;
    const int cap = t.R * (tj + 1);
    const int rows = t.TI < cap ? t.TI : cap;
    // slots [c0, TJ) on the row side, then [TJ, TJ + rows) on the column side: one contiguous walk, loaded sixteen
    // at a time (independent loads) and added one by one in slot order
    const int first = ti / t.R, last = t.TJ + rows;
    float s = 0.f;
    for (int c = first; c < last; c += 16) {
        float v[16];
#pragma unroll
        for (int u = 0; u < 16; ++u) v[u] = (c + u < last) ? p[(size_t)(c + u) * t.n_pad] : 0.f;
#pragma unroll
        for (int u = 0; u < 16; ++u)
            if (c + u < last) s += v[u];
    }
    return s;
}

// True when the whole symmetric sweep of the problem fits the tensor memory of one wave of CTAs (at most two units
// of one row block against two column blocks per SM): density and delta can then share one pass over the Gram tiles
// (launch_gram_resident).
bool gram_fits_resident(int B, int n);

// True when the resident sweep can compute the K-norm of keys with H heads of d elements on the side.
bool gram_resident_takes_knorm(int H, int d);

// One kernel for the norms, Eq. 2 and Eq. 3 on small problems: every CTA keeps the accumulators of its tiles in
// tensor memory; the diagonal tiles publish the per-token factors of their row block behind a flag that the
// density epilogues of the other tiles wait for, the grid synchronises once (bounded waits) after the density
// partials; the delta epilogue sums the partials it needs itself and re-reads the same accumulators.
// `tiling` = make_gram_tiling(n, 128).
int launch_gram_resident(const void* feat, const GramArgs& args, const GramTiling& tiling, cudaStream_t stream);

// Eq. 3 from the Gram tiles the density sweep stored: per token the nearest denser token inside the spatial radius,
// as a packed (d^2 bits, index) 64-bit minimum in args.best (reset to ~0 by the GRAM_DIAG sweep).  Bound by ALU issue
// and by the read of the tiles, not by the tensor cores.  Releases its dependents at once: a kernel that does not
// depend on it (the K-norm) can run beside it.
// `leave_room`: occupy three quarters of every SM only.
int launch_delta_pass(const GramArgs& args, const GramTiling& tiling, cudaStream_t stream, bool pdl, bool leave_room);

// Multiprocessors of the current device.
int gram_num_sms();

// Enqueues one sweep.  `tiling` must come from make_gram_tiling(n, gram_pick_bn(B, n)) for the symmetric modes.
int launch_gram_sweep(int mode, const void* feat, const GramArgs& args, const GramTiling& tiling, cudaStream_t stream,
                      bool pdl);

}  // namespace vitcop
