// Tensor-core sweep over the Gram matrix of the visual-token features (Algorithm 2, step 1) with the
// per-pair work of Eq. 2 (density) or Eq. 3 (nearest denser neighbour) fused into the epilogue.
//
// The Gram matrix f_I . f_J^T is taken on the RAW bf16 features (bf16 x bf16 products are exact in fp32) by
// tcgen05.mma with fp32 accumulators in tensor memory; the L2 normalisation enters as fp32 factors in the
// epilogue.  Nothing of size n^2 is ever written: the density sweep and the delta sweep each recompute the
// tiles they need.
//
// Symmetry: d_ij = d_ji, so the two sweeps visit only tiles that hold a pair i < j.  Such a pair serves its
// row token i (a per-thread accumulation along the row) and its column token j (a reduction over the 128
// rows of the tile: inside each warp a shuffle butterfly for the sums of Eq. 2 and one redux.sync per column for
// the minima of Eq. 3, then a fixed-order combination of the four warps that share a column range).
//
// One persistent CTA per SM, warp-specialised:
//   warp 0      TMA producer: feature tiles [128 x 64] and [BN x 64] (128-byte swizzle) into a ring of stages
//   warp 1      one thread issues tcgen05.mma (M = 128, N = BN, K = 16) into one of two TMEM accumulators
//   warps 2..   epilogue (8 warps for the density sweep, 16 for the delta sweep): warp w reads TMEM lanes
//               32 * (w % 4) .. + 31 (its rows) and one slice of the columns
// Every wait is bounded; on expiry the CTA raises an abort flag, all roles leave, TMEM is released and
// VITCOP_ERR_TIMEOUT is written to the status word.
#include <cuda.h>

#include <atomic>

#include "async_copy.cuh"
#include "gram.cuh"
#include "tcgen05.cuh"
#include "knorm.cuh"

namespace vitcop {
namespace {

constexpr int BM = kGramBM;
// Column slices an output tile is cut into for the epilogue; every slice is served by four warps (one per
// TMEM lane quarter).  The delta sweep's epilogue is the heavier one and gets twice the warps.
__host__ __device__ constexpr int epi_slices(int mode) { return mode == GRAM_DELTA ? 4 : 2; }
__host__ __device__ constexpr int gemm_threads(int mode) { return 64 + epi_slices(mode) * 128; }

// ------------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------------
// 2^x for x <= 0 (results below the normal range flush to zero); relative error about 2^-22.
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Two fp32 operations in one instruction (each half rounded like the scalar instruction): the epilogues are bound
// by instruction issue, and a pair of neighbouring columns shares every step of the distance arithmetic.
__device__ __forceinline__ unsigned long long pack2(float lo, float hi) {
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ float2 unpack2(unsigned long long v) {
    float2 o;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(o.x), "=f"(o.y) : "l"(v));
    return o;
}
__device__ __forceinline__ unsigned long long mul2(unsigned long long a, unsigned long long b) {
    unsigned long long r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ unsigned long long add2(unsigned long long a, unsigned long long b) {
    unsigned long long r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ unsigned long long fma2(unsigned long long a, unsigned long long b, unsigned long long c) {
    unsigned long long r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}

// ------------------------------------------------------------------------------------------------
// tile numbering
// ------------------------------------------------------------------------------------------------
struct KernelArgs {
    GramArgs g;
    GramTiling t;
    long long total_tiles;         // the resident sweep counts its units here
    int extra_units_per_b;         // resident sweep: units of one sample that do not hold a diagonal tile
    unsigned long long wait_ns;    // time limit of every bounded wait
    int expire_roles;              // roles whose waits give up at once: 1 load warp, 2 MMA warp, 4 epilogue warps
    __device__ __forceinline__ unsigned long long limit_of(int role) const {
        return (expire_roles & role) ? 0ull : wait_ns;
    }
};
constexpr int kRoleLoad = 1, kRoleMma = 2, kRoleEpi = 4;

template <int BN, bool SYM, bool DIAG = false>
__device__ __forceinline__ void decode_tile(const KernelArgs& k, long long t, int& b, int& ti, int& tj) {
    if (SYM) {
        decode_sym_tile(k.t, t, b, ti, tj);
        return;
    }
    b = (int)(t / k.t.tiles_per_b);
    const int r = (int)(t - (long long)b * k.t.tiles_per_b);
    if (DIAG) {
        ti = tj = r;
        return;
    }
    ti = r / k.t.TJ;
    tj = r - ti * k.t.TJ;
}

// ------------------------------------------------------------------------------------------------
// warp butterflies: lane L ends up with the reduction over the 32 lanes of element L of the array
// ------------------------------------------------------------------------------------------------
template <int HALF, bool MIN>
__device__ __forceinline__ void butterfly_stage(float* v, bool up) {
#pragma unroll
    for (int k = 0; k < HALF; ++k) {
        const float keep = up ? v[k + HALF] : v[k];
        const float send = up ? v[k] : v[k + HALF];
        const float recv = __shfl_xor_sync(0xffffffffu, send, HALF);
        v[k] = MIN ? fminf(keep, recv) : keep + recv;
    }
}
// Eight columns held by every lane (one row each): afterwards every lane holds the sum over the 32 lanes of column
// lane & 7, added in a fixed order.
__device__ __forceinline__ float warp_column_sums8(float (&v)[8], int lane) {
    butterfly_stage<4, false>(v, (lane & 4) != 0);
    butterfly_stage<2, false>(v, (lane & 2) != 0);
    butterfly_stage<1, false>(v, (lane & 1) != 0);
    float s = v[0];
    s += __shfl_xor_sync(0xffffffffu, s, 8);
    s += __shfl_xor_sync(0xffffffffu, s, 16);
    return s;
}
__device__ __forceinline__ float column_sums(float (&v)[8], int lane) { return warp_column_sums8(v, lane); }
template <bool MIN>
__device__ __forceinline__ float warp_transpose_reduce(float (&v)[32], int lane) {
    butterfly_stage<16, MIN>(v, (lane & 16) != 0);
    butterfly_stage<8, MIN>(v, (lane & 8) != 0);
    butterfly_stage<4, MIN>(v, (lane & 4) != 0);
    butterfly_stage<2, MIN>(v, (lane & 2) != 0);
    butterfly_stage<1, MIN>(v, (lane & 1) != 0);
    return v[0];
}

__device__ __forceinline__ float column_sums(float (&v)[32], int lane) { return warp_transpose_reduce<false>(v, lane); }

// ------------------------------------------------------------------------------------------------
// shared memory
// ------------------------------------------------------------------------------------------------
template <int BN>
struct GemmSmem {
    static constexpr int kStages = (BN == 128) ? 6 : 4;
    static constexpr int kABytes = BM * BK * 2;
    static constexpr int kBBytes = BN * BK * 2;
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kTileBytes = kStages * kStageBytes;
    // per column of the tile: w, a, rho, x, y; column reduction scratch: 4 x value, 4 x index;
    // row reduction scratch: 3 x value, 3 x index; per row of the tile: w, a, rho, x, y
    static constexpr int kEpiBytes = (5 + 4 + 4) * BN * 4 + (3 + 3 + 5) * BM * 4;
    static constexpr int kBarBytes = 256;
    static constexpr int kTotal = 1024 /*alignment slack*/ + kTileBytes + kEpiBytes + kBarBytes;
};

constexpr float kInf = __builtin_huge_valf();

// ------------------------------------------------------------------------------------------------
// epilogue of one output tile (called by all epilogue threads of the CTA)
// ------------------------------------------------------------------------------------------------
struct EpiSmem {
    float *colw, *cola, *colrho, *colx, *coly, *colred, *rowred;
    int *colidx, *rowidx;
    float *roww, *rowa, *rowrho, *rowx, *rowy;
    // Carves the arrays out of GemmSmem<BN>::kEpiBytes bytes at `base`.
    template <int BN>
    __device__ __forceinline__ void carve(uint8_t* base) {
        colw = reinterpret_cast<float*>(base);
        cola = colw + BN;
        colrho = cola + BN;
        colx = colrho + BN;
        coly = colx + BN;
        colred = coly + BN;                                     // [4][BN]
        colidx = reinterpret_cast<int*>(colred + 4 * BN);       // [4][BN]
        rowred = reinterpret_cast<float*>(colidx + 4 * BN);     // [3][BM]
        rowidx = reinterpret_cast<int*>(rowred + 3 * BM);       // [3][BM]
        roww = reinterpret_cast<float*>(rowidx + 3 * BM);
        rowa = roww + BM;
        rowrho = rowa + BM;
        rowx = rowrho + BM;
        rowy = rowx + BM;
    }
};
struct EpiCall {
    int b, ti, tj;                 // sample, row tile, column tile
    uint32_t tmem_tile;            // TMEM address (lane 0) of the tile's first accumulator column
    uint32_t wait_bar, wait_parity;   // mbarrier that completes when the accumulator is ready (0: it already is)
    uint32_t arrive_bar;           // mbarrier to arrive on once this thread has read the accumulator (0: none)
    bool rho_from_part;            // GRAM_DELTA: sum rho from the density partials (and publish it from diagonal tiles)
    volatile int* abort_flag;
    unsigned long long limit_ns;   // time limit of the wait for the accumulator
    float* store;                  // GRAM_RHO: where this tile's Gram values go (gram.cuh: layout), or null
};

// Returns true when the CTA must give up (a bounded wait expired somewhere).
// GW: columns a warp takes from the accumulator at a time.  32 unrolls the whole arithmetic of a 32-column chunk
// (fewest instructions; right where the code is reused tile after tile), 8 keeps it in a short rolled loop (right
// where every tile is visited once and the instruction cache would otherwise miss all the way).
template <int BN, int MODE, int METRIC, bool SPATIAL, int NS, int GW = 32>
__device__ __forceinline__ bool epi_tile(const KernelArgs& k, const EpiSmem& sm, const EpiCall& call, bool& ok) {
    static_assert(GW == 8 || GW == 32, "group width");
    constexpr bool SYM = MODE == GRAM_RHO || MODE == GRAM_DELTA;
    constexpr bool DIAG = MODE == GRAM_DIAG;
    constexpr int kEpiThreads = NS * 128;
    constexpr int kSliceCols = BN / NS;
    constexpr int kGroups = kSliceCols / GW;           // column groups per warp, taken one by one in a rolled loop
    const GramArgs& g = k.g;
    float *colw = sm.colw, *cola = sm.cola, *colrho = sm.colrho, *colx = sm.colx, *coly = sm.coly;
    float *colred = sm.colred, *rowred = sm.rowred;
    int *colidx = sm.colidx, *rowidx = sm.rowidx;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int e = threadIdx.x - 64;                    // 0 .. kEpiThreads - 1
    const int quarter = warp & 3;                      // TMEM lane quarter this warp may read
    const int slice = (warp - 2) >> 2;                 // which slice of the tile's columns this warp handles
    const int rl = quarter * 32 + lane;                // tile-local row == TMEM lane
    const int rows_out = g.row_end - g.row0;
    const int b = call.b, ti = call.ti, tj = call.tj;
    const int I0 = g.row0 + ti * BM, J0 = tj * BN;
    const int i = I0 + rl;
    const bool row_valid = SYM ? (i < g.n) : (i < g.row_end);
    const size_t bo = (size_t)b * g.n;

    // ---- per-column and per-row constants.  One item per thread where the tile allows it -- column factors,
    //      column rho and position, row factors, row rho and position -- so that all the global loads of the tile
    //      are in flight together: one round trip to L2 instead of one per group.
    const float* part_b = (MODE == GRAM_DELTA && call.rho_from_part)
                              ? g.part + (size_t)b * k.t.slots() * k.t.n_pad : nullptr;
    for (int it = e; it < 2 * BN + 2 * BM && !DIAG; it += kEpiThreads) {
        if (it < BN) {
            const int ce = it, j = J0 + ce;
            const bool cv = j < g.n;
            // (L2 loads: another CTA may have written these factors after this SM last cached their line)
            colw[ce] = cv ? __ldcg(g.w + bo + j) : 0.f;
            if (METRIC == 1) cola[ce] = cv ? __ldcg(g.a + bo + j) : 0.f;
        } else if (it < 2 * BN) {
            if (MODE == GRAM_DELTA) {
                const int ce = it - BN, j = J0 + ce;
                const bool cv = j < g.n;
                float rj = 0.f;
                float2 pj = make_float2(0.f, 0.f);
                if (cv) {
                    if (SPATIAL) pj = *reinterpret_cast<const float2*>(g.pos + 2 * (bo + j));
                    if (call.rho_from_part) {
                        rj = rho_from_partials(part_b + j, k.t, j);
                        if (ti == tj) {                        // the diagonal tile of a row block publishes its tokens' rho
                            g.rho_out[bo + j] = rj;
                            if (g.rho_user) g.rho_user[bo + j] = rj;
                        }
                    } else {
                        rj = g.rho[bo + j];
                    }
                }
                colrho[ce] = rj;
                if (SPATIAL) { colx[ce] = pj.x; coly[ce] = pj.y; }
            }
        } else if (it < 2 * BN + BM) {
            const int r = it - 2 * BN, ir = I0 + r;
            const bool rv = SYM ? (ir < g.n) : (ir < g.row_end);
            sm.roww[r] = rv ? __ldcg(g.w + bo + ir) : 0.f;
            if (METRIC == 1) sm.rowa[r] = rv ? __ldcg(g.a + bo + ir) : 0.f;
        } else if (MODE == GRAM_DELTA) {
            const int r = it - 2 * BN - BM, ir = I0 + r;
            float rr = 0.f;
            float2 pr = make_float2(0.f, 0.f);
            if (ir < g.n) {
                if (SPATIAL) pr = *reinterpret_cast<const float2*>(g.pos + 2 * (bo + ir));
                rr = call.rho_from_part ? rho_from_partials(part_b + ir, k.t, ir) : g.rho[bo + ir];
            }
            sm.rowrho[r] = rr;
            if (SPATIAL) { sm.rowx[r] = pr.x; sm.rowy[r] = pr.y; }
        }
    }
    // every pair of the tile has i < j < n: no masking needed
    const bool full = SYM && (J0 >= I0 + BM) && (J0 + BN <= g.n);

    epi_bar_sync<kEpiThreads>();
    const float w_i = DIAG ? 0.f : sm.roww[rl];
    const float a_i = METRIC == 1 ? (DIAG ? 0.f : sm.rowa[rl]) : 1.f;
    const float m2w_i = -2.f * w_i;
    float rho_i = 0.f, x_i = 0.f, y_i = 0.f;
    if (MODE == GRAM_DELTA) {
        rho_i = sm.rowrho[rl];
        if (SPATIAL) { x_i = sm.rowx[rl]; y_i = sm.rowy[rl]; }
    }
    // the row's constants, twice each, for the paired arithmetic
    const unsigned long long m2w2 = pack2(m2w_i, m2w_i), ai2 = pack2(a_i, a_i), two2 = pack2(2.f, 2.f);
    const unsigned long long nxi2 = pack2(-x_i, -x_i), nyi2 = pack2(-y_i, -y_i), c22 = pack2(g.c2, g.c2);
    if (ok && call.wait_bar) ok = mbar_wait(call.wait_bar, call.wait_parity, call.abort_flag, call.limit_ns);
    ok = __all_sync(0xffffffffu, ok);

    float racc = 0.f;                              // GRAM_RHO: row-side sum
    float rbest = kInf;                            // GRAM_DELTA: row-side minimum and its tile-local column
    int rbest_c = -1;
    if (ok) {
        tc_fence_after();
        const uint32_t taddr = call.tmem_tile + ((uint32_t)(quarter * 32) << 16) + slice * kSliceCols;
        uint32_t ld_cur[8], ld_nxt[8];
        if constexpr (GW == 8) {
            tmem_ld8_issue(taddr, ld_cur);
            tmem_ld8_wait(ld_cur);
        }
#pragma unroll 1
        for (int c = 0; c < kGroups; ++c) {
            float v[GW];
            if constexpr (GW == 8) {
                // the next group's accumulators travel while this one is worked on
                if (c + 1 < kGroups) tmem_ld8_issue(taddr + (c + 1) * 8, ld_nxt);
#pragma unroll
                for (int u = 0; u < 8; ++u) v[u] = __uint_as_float(ld_cur[u]);
            } else {
                tmem_ld32(taddr + c * 32, v);
            }
            if (c == kGroups - 1) {
                // this thread has read all it needs from the accumulator
                tc_fence_before();
                if (call.arrive_bar) mbar_arrive(call.arrive_bar);
            }
            const int cl0 = slice * kSliceCols + c * GW;       // tile-local first column of the group
            const float4* cw4 = reinterpret_cast<const float4*>(colw + cl0);
            const float4* ca4 = reinterpret_cast<const float4*>(cola + cl0);
            if (MODE == GRAM_DIAG) {
                // g_ii sits in column rl of row rl
                if (cl0 == (rl & ~(GW - 1)) && row_valid) {
                    // (selected with explicit selp: left to itself the compiler indexes the array in local
                    // memory, a cold round trip on the path every other tile waits for)
                    float gii = 0.f;
                    const int mine = lane & (GW - 1);
#pragma unroll
                    for (int u = 0; u < GW; ++u)
                        asm("{\n\t.reg .pred p;\n\tsetp.eq.s32 p, %2, %3;\n\tselp.f32 %0, %1, %0, p;\n\t}"
                            : "+f"(gii)
                            : "f"(v[u]), "r"(mine), "r"(u));
                    // The squared norm comes from the same tensor-core arithmetic as every g_ij, so the
                    // rounding of the accumulation cancels in s_ij = g_ij / sqrt(g_ii g_jj) where it
                    // matters: near-duplicates (s -> 1, d^2 = 2 - 2 s -> 0); exact duplicates give s = 1.
                    g.w_out[bo + i] = METRIC == 0 ? (gii > 0.f ? 1.0f / sqrtf(gii) : 0.f) : 1.f;
                    g.a_out[bo + i] = METRIC == 0 ? 1.f : gii;
                    if (g.best) g.best[bo + i] = ~0ull;
                }
            } else if (MODE == GRAM_SIM) {
                if (row_valid) {
                    float* o = g.sim_out + ((size_t)b * rows_out + (i - g.row0)) * g.n;
#pragma unroll
                    for (int u = 0; u < GW; ++u) {
                        const int j = J0 + cl0 + u;
                        if (j < g.n) o[j] = METRIC == 0 ? (v[u] * w_i) * colw[cl0 + u] : v[u];
                    }
                }
            } else if (MODE == GRAM_RHO) {
                if (call.store) {
                    // keep the Gram values for the delta pass: four columns of this thread's row per store, the
                    // warp's 32 rows side by side
                    float4* dst = reinterpret_cast<float4*>(call.store) + (size_t)(cl0 >> 2) * BM + rl;
#pragma unroll
                    for (int q4 = 0; q4 < GW / 4; ++q4)
                        __stcs(dst + (size_t)q4 * BM, make_float4(v[4 * q4], v[4 * q4 + 1], v[4 * q4 + 2], v[4 * q4 + 3]));
                }
                // e_ij = exp(-d_ij^2 / d_c^2), Eq. 2
#pragma unroll
                for (int q4 = 0; q4 < GW / 4; ++q4) {
                    const float4 cw = cw4[q4];
                    float4 ca = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (METRIC == 1) ca = ca4[q4];
                    if constexpr (GW == 32) {
#pragma unroll
                        for (int h = 0; h < 2; ++h) {          // two neighbouring columns at a time
                            const int u = 4 * q4 + 2 * h;
                            const unsigned long long cw2 = h ? pack2(cw.z, cw.w) : pack2(cw.x, cw.y);
                            const unsigned long long ca2 = h ? pack2(ca.z, ca.w) : pack2(ca.x, ca.y);
                            const unsigned long long x2 = mul2(pack2(v[u], v[u + 1]), cw2);
                            const unsigned long long base2 = METRIC == 0 ? two2 : add2(ai2, ca2);
                            const float2 d2 = unpack2(fma2(x2, m2w2, base2));
                            const float2 arg = unpack2(mul2(pack2(fmaxf(d2.x, 0.f), fmaxf(d2.y, 0.f)), c22));
                            v[u] = ex2_approx(arg.x);
                            v[u + 1] = ex2_approx(arg.y);
                        }
                    } else {
                        const float cwv[4] = {cw.x, cw.y, cw.z, cw.w};
                        const float cav[4] = {ca.x, ca.y, ca.z, ca.w};
#pragma unroll
                        for (int r = 0; r < 4; ++r) {
                            const int u = 4 * q4 + r;
                            const float x = v[u] * cwv[r];
                            const float base = METRIC == 0 ? 2.f : a_i + cav[r];
                            const float d2 = fmaxf(fmaf(x, m2w_i, base), 0.f);
                            v[u] = ex2_approx(d2 * g.c2);
                        }
                    }
                }
                if (!full) {
#pragma unroll
                    for (int u = 0; u < GW; ++u) {
                        const int j = J0 + cl0 + u;
                        v[u] = (j > i && j < g.n && row_valid) ? v[u] : 0.f;
                    }
                }
#pragma unroll
                for (int u = 0; u < GW; ++u) racc += v[u];
                const float cs = column_sums(v, lane);
                if (lane < GW) colred[quarter * BN + cl0 + lane] = cs;
            } else {  // GRAM_DELTA, Eq. 3
                const float4* cr4 = reinterpret_cast<const float4*>(colrho + cl0);
                const float4* cx4 = reinterpret_cast<const float4*>(colx + cl0);
                const float4* cy4 = reinterpret_cast<const float4*>(coly + cl0);
                uint32_t kc[GW];                   // column-side keys: d^2 >= 0 orders like its bit pattern
#pragma unroll
                for (int q4 = 0; q4 < GW / 4; ++q4) {
                    const float4 cw = cw4[q4];
                    const float4 cr = cr4[q4];
                    float4 ca = make_float4(0.f, 0.f, 0.f, 0.f), cx = ca, cy = ca;
                    if (METRIC == 1) ca = ca4[q4];
                    if (SPATIAL) { cx = cx4[q4]; cy = cy4[q4]; }
                    const float crv[4] = {cr.x, cr.y, cr.z, cr.w};
                    float d2v[4], s2v[4];              // squared feature distance (unclamped), squared spatial distance
                    if constexpr (GW == 32) {
#pragma unroll
                        for (int h = 0; h < 2; ++h) {          // two neighbouring columns at a time
                            const int u = 4 * q4 + 2 * h;
                            const unsigned long long cw2 = h ? pack2(cw.z, cw.w) : pack2(cw.x, cw.y);
                            const unsigned long long ca2 = h ? pack2(ca.z, ca.w) : pack2(ca.x, ca.y);
                            const unsigned long long x2 = mul2(pack2(v[u], v[u + 1]), cw2);
                            const unsigned long long base2 = METRIC == 0 ? two2 : add2(ai2, ca2);
                            const float2 d2 = unpack2(fma2(x2, m2w2, base2));
                            d2v[2 * h] = d2.x;
                            d2v[2 * h + 1] = d2.y;
                            if (SPATIAL) {
                                const unsigned long long dx2 = add2(h ? pack2(cx.z, cx.w) : pack2(cx.x, cx.y), nxi2);
                                const unsigned long long dy2 = add2(h ? pack2(cy.z, cy.w) : pack2(cy.x, cy.y), nyi2);
                                const float2 s2 = unpack2(fma2(dx2, dx2, mul2(dy2, dy2)));
                                s2v[2 * h] = s2.x;
                                s2v[2 * h + 1] = s2.y;
                            }
                        }
                    } else {
                        const float cwv[4] = {cw.x, cw.y, cw.z, cw.w};
                        const float cav[4] = {ca.x, ca.y, ca.z, ca.w};
                        const float cxv[4] = {cx.x, cx.y, cx.z, cx.w};
                        const float cyv[4] = {cy.x, cy.y, cy.z, cy.w};
#pragma unroll
                        for (int r = 0; r < 4; ++r) {
                            const float x = v[4 * q4 + r] * cwv[r];
                            d2v[r] = fmaf(x, m2w_i, METRIC == 0 ? 2.f : a_i + cav[r]);
                            if (SPATIAL) {
                                const float dx = cxv[r] - x_i, dy = cyv[r] - y_i;
                                s2v[r] = fmaf(dx, dx, dy * dy);
                            }
                        }
                    }
#pragma unroll
                    for (int r = 0; r < 4; ++r) {
                        const int u = 4 * q4 + r;
                        float d2 = fmaxf(d2v[r], 0.f);
                        bool usable = true;        // the pair may serve as (child, parent) at all
                        if (SPATIAL) usable = s2v[r] <= g.tau2;
                        if (!full) {
                            const int j = J0 + cl0 + u;
                            usable = usable && j > i && j < g.n && row_valid;
                        }
                        if (SPATIAL || !full) d2 = usable ? d2 : kInf;
                        // with i < j: "j denser than i" is rho_j > rho_i, "i denser than j" is its complement
                        const bool jd = crv[r] > rho_i;
                        const float kr = jd ? d2 : kInf;       // j as parent candidate of i (row side)
                        kc[u] = __float_as_uint(jd ? kInf : d2);   // i as parent candidate of j (column side)
                        if (kr < rbest) { rbest = kr; rbest_c = cl0 + u; }
                    }
                }
                // column side: minimum over this warp's 32 rows and the lowest row that attains it
                uint32_t my_min = 0x7f800000u, my_rows = 0;
#pragma unroll
                for (int u = 0; u < GW; ++u) {
                    const uint32_t m = __reduce_min_sync(0xffffffffu, kc[u]);
                    const uint32_t rows = __ballot_sync(0xffffffffu, kc[u] == m);
                    if (lane == u) { my_min = m; my_rows = rows; }
                }
                if (lane < GW) {
                    colred[quarter * BN + cl0 + lane] = __uint_as_float(my_min);
                    colidx[quarter * BN + cl0 + lane] =
                        my_min < 0x7f800000u ? I0 + quarter * 32 + (__ffs(my_rows) - 1) : -1;
                }
            }
            if constexpr (GW == 8) {
                if (c + 1 < kGroups) {
                    tmem_ld8_wait(ld_nxt);
#pragma unroll
                    for (int u = 0; u < 8; ++u) ld_cur[u] = ld_nxt[u];
                }
            }
        }
    }

    if (MODE == GRAM_DIAG && g.bbox) {
        // ---- bounding box of the row block's positions: per warp by shuffles, the four row quarters through shared
        //      memory (rows outside the sample and coordinates that are not numbers leave the box alone)
        if (slice == 0) {
            float4 bx = make_float4(kInf, kInf, -kInf, -kInf);
            if (row_valid) {
                const float2 q = *reinterpret_cast<const float2*>(g.pos + 2 * (bo + i));
                bx = make_float4(q.x, q.y, q.x, q.y);
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
                bx.x = fminf(bx.x, __shfl_xor_sync(0xffffffffu, bx.x, off));
                bx.y = fminf(bx.y, __shfl_xor_sync(0xffffffffu, bx.y, off));
                bx.z = fmaxf(bx.z, __shfl_xor_sync(0xffffffffu, bx.z, off));
                bx.w = fmaxf(bx.w, __shfl_xor_sync(0xffffffffu, bx.w, off));
            }
            if (lane == 0) reinterpret_cast<float4*>(rowred)[quarter] = bx;
        }
        epi_bar_sync<kEpiThreads>();
        if (e == 0 && ok) {
            float4 bx = reinterpret_cast<const float4*>(rowred)[0];
#pragma unroll
            for (int q = 1; q < 4; ++q) {
                const float4 o = reinterpret_cast<const float4*>(rowred)[q];
                bx = make_float4(fminf(bx.x, o.x), fminf(bx.y, o.y), fmaxf(bx.z, o.z), fmaxf(bx.w, o.w));
            }
            g.bbox[(size_t)b * k.t.TI + ti] = bx;
        }
    }
    if (SYM) {
        // ---- combine the four column slices of every row and the four row quarters of every column
        if (slice > 0) {
            rowred[(slice - 1) * BM + rl] = MODE == GRAM_RHO ? racc : rbest;
            if (MODE == GRAM_DELTA) rowidx[(slice - 1) * BM + rl] = rbest_c;
        }
        epi_bar_sync<kEpiThreads>();
        if (ok) {
            const int slot_base = b * k.t.slots();
            if (MODE == GRAM_RHO) {
                if (slice == 0 && row_valid) {
#pragma unroll
                    for (int q = 0; q < NS - 1; ++q) racc += rowred[q * BM + rl];       // fixed order
                    g.part[((size_t)(slot_base + tj)) * k.t.n_pad + i] = racc;
                }
                for (int ce = e; ce < BN; ce += kEpiThreads)
                    if (J0 + ce < g.n)
                        g.part[((size_t)(slot_base + k.t.TJ + ti)) * k.t.n_pad + J0 + ce] =
                            ((colred[ce] + colred[BN + ce]) + colred[2 * BN + ce]) + colred[3 * BN + ce];
            } else {
                if (slice == 0 && row_valid) {
#pragma unroll
                    for (int q = 0; q < NS - 1; ++q) {                             // ascending columns: ties keep the lower one
                        const float other = rowred[q * BM + rl];
                        if (other < rbest) { rbest = other; rbest_c = rowidx[q * BM + rl]; }
                    }
                    if (rbest_c >= 0) {
                        const unsigned long long packed =
                            ((unsigned long long)__float_as_uint(rbest) << 32) |
                            (unsigned long long)(uint32_t)(J0 + rbest_c);
                        atomicMin(g.best + bo + i, packed);
                    }
                }
                for (int ce = e; ce < BN; ce += kEpiThreads) {
                    if (J0 + ce >= g.n) continue;
                    float bk = kInf;
                    int bi = -1;
#pragma unroll
                    for (int q = 0; q < 4; ++q) {                                  // ascending rows: ties keep the lower row
                        const float kk = colred[q * BN + ce];
                        if (kk < bk) { bk = kk; bi = colidx[q * BN + ce]; }
                    }
                    if (bi >= 0) {
                        const unsigned long long packed =
                            ((unsigned long long)__float_as_uint(bk) << 32) | (unsigned long long)(uint32_t)bi;
                        atomicMin(g.best + bo + J0 + ce, packed);
                    }
                }
            }
        }
    }
    // shared arrays are rewritten for the next tile; all epilogue warps leave together or not at all
    return epi_bar_or<kEpiThreads>(!ok);
}

// ------------------------------------------------------------------------------------------------
// the kernel
// ------------------------------------------------------------------------------------------------
template <int BN, int MODE, int METRIC, bool SPATIAL>
__global__ void __launch_bounds__(gemm_threads(MODE), 1)
gram_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const KernelArgs k) {
    using S = GemmSmem<BN>;
    constexpr bool SYM = MODE == GRAM_RHO || MODE == GRAM_DELTA;
    constexpr bool DIAG = MODE == GRAM_DIAG;            // BN == BM: a diagonal tile multiplies the row block by itself
    constexpr int NS = epi_slices(MODE);
    constexpr int kEpiThreads = NS * 128;
    const GramArgs& g = k.g;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;                 // 1024-byte aligned for the 128B swizzle
    uint8_t* gen = smem_raw + (tiles - raw);
    EpiSmem sm;
    sm.template carve<BN>(gen + S::kTileBytes);
    uint64_t* bars = reinterpret_cast<uint64_t*>(gen + S::kTileBytes + S::kEpiBytes);
    // barriers: full[kStages], empty[kStages], tmem_full[2], tmem_empty[2], drain
    const uint32_t bar_full = smem_u32(bars);
    const uint32_t bar_empty = bar_full + 8 * S::kStages;
    const uint32_t bar_tfull = bar_empty + 8 * S::kStages;
    const uint32_t bar_tempty = bar_tfull + 16;
    const uint32_t bar_drain = bar_tempty + 16;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * S::kStages + 5);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    // (the last words of the barrier block hold the epilogue's mask of tiles that are not kept)
    static_assert((2 * S::kStages + 5) * 8 + 8 + (NS * 128 / 32) * 4 <= S::kBarBytes, "barrier block too small");

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr uint32_t kTmemCols = 2 * BN;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S::kStages; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(bar_tfull + 8 * a, 1);
            mbar_init(bar_tempty + 8 * a, kEpiThreads);   // every epilogue thread arrives once per tile
        }
        mbar_init(bar_drain, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_a)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_b)) : "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // The kernels that follow on the stream may be scheduled from here on; they wait for this grid to complete
    // before they touch anything it writes.  A density sweep that has a kernel running beside it (filter.cu: the list
    // of tiles within the spatial radius) releases them only once its own predecessors are complete, so that the
    // neighbour may rely on their results without a wait of its own.
    const bool release_late = MODE == GRAM_RHO && g.bbox != nullptr;
    if (!release_late) grid_dependency_launch_dependents();

    const long long total_tiles = k.total_tiles;
    const int KB = g.D / BK;
    uint32_t issued = 0, issued_parity = 0;    // thread 0, per stage: a load was issued / parity of its phase

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        // The features are an input of the whole call (never written by the kernel before this one), so
        // the loads need not wait for the preceding grid.
        if (lane == 0) {
            const unsigned long long lim = k.limit_of(kRoleLoad);
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            for (long long t = blockIdx.x; ok && t < total_tiles; t += gridDim.x) {
                int b, ti, tj;
                decode_tile<BN, SYM, DIAG>(k, t, b, ti, tj);
                const int I0 = g.row0 + ti * BM, J0 = tj * BN;
                for (int kb = 0; kb < KB; ++kb) {
                    if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, lim)) { ok = false; break; }
                    const uint32_t sa = tiles + stage * S::kStageBytes;
                    mbar_expect_tx(bar_full + 8 * stage, DIAG ? S::kABytes : S::kStageBytes);
                    tma_load_3d(sa, &map_a, bar_full + 8 * stage, kb * BK, I0, b);
                    if (!DIAG) tma_load_3d(sa + S::kABytes, &map_b, bar_full + 8 * stage, kb * BK, J0, b);
                    issued |= 1u << stage;
                    issued_parity = (issued_parity & ~(1u << stage)) | (phase << stage);
                    if (++stage == S::kStages) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(BM, BN);
            const unsigned long long lim = k.limit_of(kRoleMma);
            uint32_t stage = 0, phase = 0;
            uint32_t acc = 0, acc_phase = 0;
            bool ok = true;
            for (long long t = blockIdx.x; ok && t < total_tiles; t += gridDim.x) {
                if (!mbar_wait(bar_tempty + 8 * acc, acc_phase ^ 1u, abort_flag, lim)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * BN;
                for (int kb = 0; kb < KB; ++kb) {
                    if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag, lim)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = tiles + stage * S::kStageBytes;
                    const uint64_t da = umma_desc_k128(sa), db = DIAG ? da : umma_desc_k128(sa + S::kABytes);
#pragma unroll
                    for (int kk = 0; kk < BK / UMMA_K; ++kk) {
                        // advancing 16 elements (32 bytes) along K inside the swizzle row: +2 in address units
                        tc_mma_bf16(d_tmem, da + (uint64_t)(2 * kk), db + (uint64_t)(2 * kk), idesc,
                                    (kb > 0 || kk > 0) ? 1u : 0u);
                    }
                    tc_commit(bar_empty + 8 * stage);      // frees the smem stage once these MMAs have read it
                    if (++stage == S::kStages) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                tc_commit(bar_tfull + 8 * acc);            // accumulator complete
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
            if (!ok) {
                // leaving early: let the MMAs already issued finish before TMEM is released
                tc_commit(bar_drain);
                mbar_drain(bar_drain, 0);
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2 ..)
        uint32_t acc = 0, acc_phase = 0;
        bool ok = true;
        const bool skip_far = MODE == GRAM_RHO && g.gram_tiles && g.bbox;
        uint32_t* far_mask = reinterpret_cast<uint32_t*>(reinterpret_cast<uint8_t*>(bars) + S::kBarBytes) - kEpiThreads / 32;
        long long kt = 0;                                  // tiles this CTA has taken

        grid_dependency_wait();                            // w, a, rho, best come from the preceding kernels
        if (release_late) grid_dependency_launch_dependents();

        for (long long t = blockIdx.x; t < total_tiles; t += gridDim.x) {
            EpiCall c;
            decode_tile<BN, SYM, DIAG>(k, t, c.b, c.ti, c.tj);
            c.tmem_tile = tmem_base + acc * BN;
            c.wait_bar = bar_tfull + 8 * acc;
            c.wait_parity = acc_phase;
            c.arrive_bar = bar_tempty + 8 * acc;
            c.rho_from_part = false;
            c.abort_flag = abort_flag;
            c.limit_ns = k.limit_of(kRoleEpi);
            c.store = (MODE == GRAM_RHO && g.gram_tiles) ? g.gram_tiles + (size_t)t * gram_tile_floats(BN) : nullptr;
            if (skip_far) {
                // a tile beyond the spatial radius is of no use to Eq. 3 and is not kept (gram.cuh:
                // tile_outside_radius); the CTA's next kEpiThreads tiles are tested together, one per thread
                const int kk = (int)(kt % kEpiThreads);
                if (kk == 0) {
                    epi_bar_sync<kEpiThreads>();               // (the previous mask has been read by everyone)
                    const long long mine = t + (long long)(threadIdx.x - 64) * gridDim.x;
                    bool far = false;
                    if (mine < total_tiles) {
                        int fb, fti, ftj;
                        decode_tile<BN, SYM, DIAG>(k, mine, fb, fti, ftj);
                        far = tile_outside_radius(g.bbox + (size_t)fb * k.t.TI, k.t, fti, ftj, g.tau2);
                    }
                    const uint32_t bal = __ballot_sync(0xffffffffu, far);
                    if (lane == 0) far_mask[warp - 2] = bal;
                    epi_bar_sync<kEpiThreads>();
                }
                if (far_mask[kk >> 5] >> (kk & 31) & 1u) c.store = nullptr;
            }
            ++kt;
            if (epi_tile<BN, MODE, METRIC, SPATIAL, NS>(k, sm, c, ok)) break;
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
    if (threadIdx.x == 0 && *abort_flag) {
        // Some role gave up, so loads this thread issued may never have been consumed: give the copies still in
        // flight into this CTA's shared memory time to land before the CTA goes away.
        for (int s = 0; s < S::kStages; ++s)
            if (issued >> s & 1u) mbar_drain(bar_full + 8 * s, issued_parity >> s & 1u);
        if (g.status) atomicMax(g.status, VITCOP_ERR_TIMEOUT);
    }
}


// ------------------------------------------------------------------------------------------------
// the resident kernel: density and delta from ONE pass over the Gram tiles (small problems)
// ------------------------------------------------------------------------------------------------
// The unit of work is one row block (128 tokens) against two adjacent column blocks: one MMA of N = 256 per
// k-step, the row operand loaded once for both 128 x 128 tiles (a quarter less operand traffic than tile by tile,
// and the tensor cores run N = 256 at twice the rate of N = 128).  Row block ti owns the column blocks ti .. TI - 1,
// paired from the diagonal on; the last unit of a row is half empty when their number is odd (the rows of its
// missing column block lie outside the tensor and are zero-filled at no cost in traffic).  A CTA owns at most
// kResidentUnits units and keeps their accumulators in tensor memory (2 x 256 of the 512 columns).  Units that
// start with a diagonal tile are numbered first, so that these accumulators are the first to complete.
// Phases of the epilogue warps, which treat a unit as two tiles of 128 x 128:
//   0. the diagonal tiles yield g_ii -> per-token normalisation factors, published behind one flag per row block
//   1. density epilogue of every tile (after the flags of its row and column block) -> rho partials;
//      grid-wide barrier
//   2. delta epilogue of every tile, re-reading the accumulators; rho of the tile's rows and columns is summed
//      from the partials on the way (the diagonal tiles publish it)
// The grid (at most one CTA per SM) is launched cooperatively, so all CTAs are resident together; flags and barrier
// are words in global memory with bounded waits.  No wait can form a cycle: a flag is raised by a CTA that has
// waited for nothing but its own tensor-core work.
// The load warp and the MMA warp are idle once the CTA's last MMA is issued, and so are, a little later, the
// operand buffers and -- for the rest of the kernel, which is arithmetic on the accumulators -- the memory system:
// if the caller has a K-norm (Eq. 4) to compute, these two warps stream K through the operand buffers with bulk
// copies and reduce it there (resident_knorm).
constexpr int kResidentUnits = 2;
constexpr int kResidentBN = 2 * BM;                       // columns of a unit
constexpr int kResidentEpiThreads = 512;

__device__ __forceinline__ unsigned int ld_acquire_u32(const unsigned int* p) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Barrier over all CTAs of the grid, called by the epilogue threads.  Returns true when the grid must give up.
// One thread speaks for the CTA: the CTA barrier orders every epilogue thread's writes before that thread's fence
// (and its fence before their later reads), so the other threads need none of their own.
__device__ __forceinline__ bool resident_grid_barrier(unsigned int* counter, volatile int* abort_flag, bool aborted,
                                                      unsigned long long limit_ns) {
    epi_bar_sync<kResidentEpiThreads>();
    if (threadIdx.x == 64 && !aborted) {
        __threadfence();
        atomicAdd(counter, 1u);
        const unsigned long long t0 = global_ns();
        while (ld_acquire_u32(counter) < gridDim.x) {
            if (limit_ns == 0ull || global_ns() - t0 > limit_ns) { *abort_flag = 1; break; }
        }
        __threadfence();
    }
    return epi_bar_or<kResidentEpiThreads>(aborted || *abort_flag != 0);
}

// Raises a flag once every epilogue thread's global writes are visible device-wide.
__device__ __forceinline__ void resident_publish(unsigned int* flag) {
    epi_bar_sync<kResidentEpiThreads>();
    if (threadIdx.x == 64) {
        __threadfence();
        asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(flag), "r"(1u) : "memory");
    }
}

// Waits (bounded) until both flags are up.  Returns true when the grid must give up.
__device__ __forceinline__ bool resident_wait_flags(const unsigned int* fa, const unsigned int* fb,
                                                    volatile int* abort_flag, bool aborted, unsigned long long limit_ns) {
    if (threadIdx.x == 64 && !aborted) {
        const unsigned long long t0 = global_ns();
        while (ld_acquire_u32(fa) == 0u || ld_acquire_u32(fb) == 0u) {
            if (limit_ns == 0ull || global_ns() - t0 > limit_ns) { *abort_flag = 1; break; }
        }
        __threadfence();
    }
    return epi_bar_or<kResidentEpiThreads>(aborted || *abort_flag != 0);
}

// Unit t of the resident sweep: the B * TI units that start with a diagonal tile first, then the others, sample
// by sample and row block by row block.
struct ResidentUnit {
    int b, ti, tj0;        // sample, row block, first column block
    int width;             // column blocks inside the tensor: 2, or 1 for the half-empty last unit of a row
};
__host__ __device__ inline int resident_extra_units(int TI) {
    int e = 0;
    for (int ti = 0; ti < TI; ++ti) e += (TI - ti + 1) / 2 - 1;
    return e;
}
__device__ __forceinline__ ResidentUnit decode_resident_unit(const KernelArgs& k, long long t) {
    const int TI = k.t.TI;
    const long long n_diag = (long long)k.g.B * TI;
    ResidentUnit u;
    if (t < n_diag) {
        u.b = (int)(t / TI);
        u.ti = (int)(t - (long long)u.b * TI);
        u.tj0 = u.ti;
    } else {
        const long long x = t - n_diag;                    // extra_units_per_b > 0 here
        u.b = (int)(x / k.extra_units_per_b);
        int r = (int)(x - (long long)u.b * k.extra_units_per_b);
        int ti = 0;
        for (; ti < TI; ++ti) {
            const int m = (TI - ti + 1) / 2 - 1;           // units of row block ti beyond its first
            if (r < m) break;
            r -= m;
        }
        u.ti = ti;
        u.tj0 = ti + 2 * (r + 1);
    }
    u.width = u.tj0 + 1 < TI ? 2 : 1;
    return u;
}

constexpr int kKnChunkTokens = 8;                          // tokens per chunk: 8 threads each
constexpr int kKnBuffers = 3;

// K-norm (Eq. 4) by the 64 threads of warps 0 and 1, after the CTA's last MMA has completed.  Chunks of eight
// consecutive tokens of one sample are copied head by head (one contiguous run per head) into the operand
// buffers, up to three chunks in flight; eight threads reduce one token, each standing in for lanes s and s + 8
// of the sixteen-lane reduction of the stand-alone kernel, so that both give the same bits.
__device__ __forceinline__ void resident_knorm(const GramArgs& g, const uint8_t* buf_gen, uint32_t buf_smem,
                                               uint32_t buf_bytes, uint32_t bar_kn, uint32_t bar_last_mma,
                                               volatile int* abort_flag, unsigned long long limit_ns) {
    const int tid = threadIdx.x;                           // 0 .. 63
    auto all_ok = [](bool ok) {
        uint32_t out;
        asm volatile(
            "{\n\t.reg .pred p, q;\n\t"
            "setp.eq.b32 p, %1, 0;\n\t"
            "bar.red.or.pred q, 2, 64, p;\n\t"
            "selp.u32 %0, 0, 1, q;\n\t}"
            : "=r"(out) : "r"((uint32_t)ok) : "memory");
        return out != 0;
    };
    // the tensor cores read the operand buffers until the last MMA completes
    if (!all_ok(mbar_wait(bar_last_mma, 0, abort_flag, limit_ns))) return;

    const int H = g.kn_H, d8 = g.kn_d / 8, Nv = g.kn_Nv;
    const uint32_t row_bytes = (uint32_t)d8 * 16u;
    const uint32_t head_bytes = kKnChunkTokens * row_bytes;         // one head of a chunk
    const uint32_t chunk_bytes = (uint32_t)H * head_bytes;
    const int nbuf = min(kKnBuffers, (int)(buf_bytes / chunk_bytes));   // >= 1 (gram_resident_takes_knorm)
    const int chunks_per_b = (Nv + kKnChunkTokens - 1) / kKnChunkTokens;
    const long long total = (long long)g.kn_B * chunks_per_b;
    const uint8_t* Kb = static_cast<const uint8_t*>(g.kn_K);
    const size_t head_stride = (size_t)g.kn_N * row_bytes;

    auto issue = [&](long long c, int buf) {               // thread 0
        const int b = (int)(c / chunks_per_b);
        const int i0 = (int)(c - (long long)b * chunks_per_b) * kKnChunkTokens;
        const int cnt = min(kKnChunkTokens, Nv - i0);
        const uint32_t run = (uint32_t)cnt * row_bytes;
        mbar_expect_tx(bar_kn + 8 * buf, (uint32_t)H * run);
        const uint8_t* src = Kb + ((size_t)b * H * g.kn_N + (size_t)(g.kn_vis_start + i0)) * row_bytes;
        const uint32_t dst = buf_smem + (uint32_t)buf * chunk_bytes;
        for (int h = 0; h < H; ++h) bulk_load(dst + (uint32_t)h * head_bytes, src + (size_t)h * head_stride, run, bar_kn + 8 * buf);
    };
    long long issued = 0;                                  // chunks this CTA has requested (thread 0)
    if (tid == 0)
        for (; issued < nbuf && blockIdx.x + issued * gridDim.x < total; ++issued)
            issue(blockIdx.x + issued * gridDim.x, (int)issued);

    const int tk = tid >> 3, s = tid & 7;
    long long it = 0;
    bool ok = true;
    for (long long c = blockIdx.x; c < total; c += gridDim.x, ++it) {
        const int buf = (int)(it % nbuf);
        ok = all_ok(mbar_wait(bar_kn + 8 * buf, (uint32_t)((it / nbuf) & 1), abort_flag, limit_ns));
        if (!ok) break;
        const int b = (int)(c / chunks_per_b);
        const int i0 = (int)(c - (long long)b * chunks_per_b) * kKnChunkTokens;
        const int cnt = min(kKnChunkTokens, Nv - i0);
        const uint4* rows = reinterpret_cast<const uint4*>(buf_gen + (size_t)buf * chunk_bytes) + (size_t)tk * d8;
        const int head16 = kKnChunkTokens * d8;            // uint4 per head of a chunk
        float part = 0.f;
        if (tk < cnt) {
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                float a0 = 0.f, a1 = 0.f;
                for (int piece = s + 8 * q; piece < d8; piece += 16) {
#pragma unroll 8
                    for (int h = 0; h < H; ++h) knorm_sq_acc(rows[(size_t)h * head16 + piece], a0, a1);
                }
                part += a0 + a1;
            }
        }
#pragma unroll
        for (int off = 4; off > 0; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
        if (tk < cnt && s == 0) g.kn_score[(size_t)b * Nv + i0 + tk] = sqrtf(part);
        asm volatile("bar.sync 2, 64;" ::: "memory");      // the buffer has been read by everyone
        if (tid == 0) {
            const long long cn = blockIdx.x + issued * gridDim.x;
            if (cn < total) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                issue(cn, buf);
                ++issued;
            }
        }
    }
    if (!ok && tid == 0) {
        // giving up: wait (bounded) for the copies still in flight before the CTA's shared memory goes away
        for (long long j = it; j < issued; ++j) mbar_drain(bar_kn + 8 * (int)(j % nbuf), (uint32_t)((j / nbuf) & 1));
    }
}

template <int METRIC, bool SPATIAL>
__global__ void __launch_bounds__(64 + kResidentEpiThreads, 1)
gram_resident_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                     const KernelArgs k) {
    constexpr int BN = BM;                                 // the epilogue's tiles
    constexpr int NS = 4;
    using S = GemmSmem<kResidentBN>;                       // stages of 128 + 256 operand rows
    const GramArgs& g = k.g;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;
    uint8_t* gen = smem_raw + (tiles - raw);
    EpiSmem sm;
    sm.template carve<BN>(gen + S::kTileBytes);
    uint64_t* bars = reinterpret_cast<uint64_t*>(gen + S::kTileBytes + S::kEpiBytes);
    // barriers: full[kStages], empty[kStages], tmem_full[kResidentUnits], drain, knorm[kKnBuffers]
    const uint32_t bar_full = smem_u32(bars);
    const uint32_t bar_empty = bar_full + 8 * S::kStages;
    const uint32_t bar_tfull = bar_empty + 8 * S::kStages;
    const uint32_t bar_drain = bar_tfull + 8 * kResidentUnits;
    const uint32_t bar_kn = bar_drain + 8;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * S::kStages + kResidentUnits + 1 + kKnBuffers);
    static_assert((2 * S::kStages + kResidentUnits + 1 + kKnBuffers) * 8 + 8 <= S::kBarBytes, "barrier block too small");
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr uint32_t kTmemCols = kResidentUnits * kResidentBN;   // 512: the whole tensor memory of the SM

    if (threadIdx.x == 0) {
        for (int s = 0; s < S::kStages; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int a = 0; a < kResidentUnits; ++a) mbar_init(bar_tfull + 8 * a, 1);
        mbar_init(bar_drain, 1);
        for (int a = 0; a < kKnBuffers; ++a) mbar_init(bar_kn + 8 * a, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_a)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_b)) : "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const long long total_units = k.total_tiles;          // <= kResidentUnits * gridDim.x (checked by the launcher)
    const int KB = g.D / BK;
    uint32_t issued = 0, issued_parity = 0;               // thread 0, per stage: a load was issued / parity of its phase

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const unsigned long long lim = k.limit_of(kRoleLoad);
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            for (long long t = blockIdx.x; ok && t < total_units; t += gridDim.x) {
                const ResidentUnit u = decode_resident_unit(k, t);
                const int I0 = u.ti * BM, J0 = u.tj0 * BM;
                for (int kb = 0; kb < KB; ++kb) {
                    if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, lim)) { ok = false; break; }
                    const uint32_t sa = tiles + stage * S::kStageBytes;
                    // rows of the box past the sample's last token are zero-filled and still count as received
                    mbar_expect_tx(bar_full + 8 * stage, S::kStageBytes);
                    tma_load_3d(sa, &map_a, bar_full + 8 * stage, kb * BK, I0, u.b);
                    tma_load_3d(sa + S::kABytes, &map_b, bar_full + 8 * stage, kb * BK, J0, u.b);
                    issued |= 1u << stage;
                    issued_parity = (issued_parity & ~(1u << stage)) | (phase << stage);
                    if (++stage == S::kStages) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer: unit s of this CTA -> columns 256 s ..
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(BM, kResidentBN);
            const unsigned long long lim = k.limit_of(kRoleMma);
            uint32_t stage = 0, phase = 0;
            uint32_t slot = 0;
            bool ok = true;
            for (long long t = blockIdx.x; ok && t < total_units; t += gridDim.x, ++slot) {
                const uint32_t d_tmem = tmem_base + slot * kResidentBN;
                for (int kb = 0; kb < KB; ++kb) {
                    if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag, lim)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = tiles + stage * S::kStageBytes;
                    const uint64_t da = umma_desc_k128(sa), db = umma_desc_k128(sa + S::kABytes);
#pragma unroll
                    for (int kk = 0; kk < BK / UMMA_K; ++kk)
                        tc_mma_bf16(d_tmem, da + (uint64_t)(2 * kk), db + (uint64_t)(2 * kk), idesc,
                                    (kb > 0 || kk > 0) ? 1u : 0u);
                    tc_commit(bar_empty + 8 * stage);
                    if (++stage == S::kStages) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                tc_commit(bar_tfull + 8 * slot);
            }
            if (!ok) {
                tc_commit(bar_drain);
                mbar_drain(bar_drain, 0);
            }
        }
    }
    if (warp < 2) {
        __syncwarp();
        if (g.kn_K) {
            const long long my_units = (total_units - blockIdx.x + gridDim.x - 1) / gridDim.x;   // >= 1
            resident_knorm(g, gen, tiles, (uint32_t)S::kTileBytes, bar_kn, bar_tfull + 8 * (uint32_t)(my_units - 1),
                           abort_flag, k.limit_of(kRoleLoad | kRoleMma));
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..17)
        bool ok = true;
        bool stop = false;
        const unsigned long long lim = k.limit_of(kRoleEpi);
        grid_dependency_wait();
        // tile s (0 or 1) of this CTA's unit number `slot`
        auto tile_call = [&](const ResidentUnit& u, uint32_t slot, int s, bool wait_mma, bool rho_from_part) {
            EpiCall c;
            c.b = u.b;
            c.ti = u.ti;
            c.tj = u.tj0 + s;
            c.tmem_tile = tmem_base + slot * kResidentBN + (uint32_t)s * BN;
            c.wait_bar = wait_mma ? bar_tfull + 8 * slot : 0;
            c.wait_parity = 0;
            c.arrive_bar = 0;
            c.rho_from_part = rho_from_part;
            c.abort_flag = abort_flag;
            c.limit_ns = lim;
            c.store = nullptr;
            return c;
        };

        // ---- phase 0: the diagonal tiles give g_ii, hence the per-token factors every other epilogue needs
        uint32_t slot = 0;
        for (long long t = blockIdx.x; t < total_units && !stop; t += gridDim.x, ++slot) {
            const ResidentUnit u = decode_resident_unit(k, t);
            if (u.ti != u.tj0) continue;                   // uniform over the CTA
            const EpiCall c = tile_call(u, slot, 0, true, false);
            stop = epi_tile<BN, GRAM_DIAG, METRIC, false, NS, 8>(k, sm, c, ok);
            if (!stop) resident_publish(g.diag_ready + (size_t)u.b * k.t.TI + u.ti);
        }
        // ---- phase 1: density partials, tile by tile as soon as the factors of its row and column block exist
        slot = 0;
        for (long long t = blockIdx.x; t < total_units && !stop; t += gridDim.x, ++slot) {
            const ResidentUnit u = decode_resident_unit(k, t);
            for (int s = 0; s < u.width && !stop; ++s) {
                const EpiCall c = tile_call(u, slot, s, true, false);
                if (c.ti != c.tj)
                    stop = resident_wait_flags(g.diag_ready + (size_t)c.b * k.t.TI + c.ti,
                                               g.diag_ready + (size_t)c.b * k.t.TI + c.tj, abort_flag, stop, lim);
                if (!stop) stop = epi_tile<BN, GRAM_RHO, METRIC, false, NS, 8>(k, sm, c, ok);
            }
        }
        stop = resident_grid_barrier(g.grid_sync, abort_flag, stop, lim);
        // The kernels that follow cannot share an SM with a CTA of this grid (registers, shared memory); from here
        // on they may at least be set up.
        grid_dependency_launch_dependents();
        // ---- phase 2: delta and parents from the same accumulators; every tile sums the rho of its own rows and
        //      columns from the partials (fixed order: the same bits everywhere)
        slot = 0;
        for (long long t = blockIdx.x; t < total_units && !stop; t += gridDim.x, ++slot) {
            const ResidentUnit u = decode_resident_unit(k, t);
            for (int s = 0; s < u.width && !stop; ++s) {
                const EpiCall c = tile_call(u, slot, s, false, true);
                stop = epi_tile<BN, GRAM_DELTA, METRIC, SPATIAL, NS, 8>(k, sm, c, ok);
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
    if (threadIdx.x == 0 && *abort_flag) {
        // (see gram_tc_kernel: unconsumed operand loads must have landed before the CTA goes away)
        for (int s = 0; s < S::kStages; ++s)
            if (issued >> s & 1u) mbar_drain(bar_full + 8 * s, issued_parity >> s & 1u);
        if (g.status) atomicMax(g.status, VITCOP_ERR_TIMEOUT);
    }
    grid_dependency_launch_dependents();
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// 3-D view (D, n, B) of the bf16 feature tensor with a (64, box_rows, 1) box and the 128-byte swizzle.
bool make_feat_map(CUtensorMap* map, const void* feat, int B, int n, int D, int box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)n, (cuuint64_t)B};
    cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)n * D * 2};
    cuuint32_t box[3] = {(cuuint32_t)BK, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(feat), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Time limit of the kernels' bounded waits and, for failure-handling tests, the roles whose waits give up at once.
std::atomic<unsigned long long> g_wait_ns{kWaitLimitNs};
std::atomic<int> g_expire_roles{0};

// What the launchers remember is remembered per device: one process may drive several.
constexpr int kMaxDevices = 64;
int current_device() {
    int dev = 0;
    return (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < kMaxDevices) ? dev : 0;
}

int num_sms() {
    static std::atomic<int> sms[kMaxDevices];
    const int dev = current_device();
    int v = sms[dev].load(std::memory_order_relaxed);
    if (v <= 0) {
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) v = 148;
        sms[dev].store(v, std::memory_order_relaxed);
    }
    return v;
}

// Raises a kernel's dynamic shared-memory limit once per device.
template <typename Kernel>
int allow_dynamic_smem(Kernel kern, int bytes, std::atomic<unsigned long long>& done) {
    const unsigned long long bit = 1ull << current_device();
    if (done.load(std::memory_order_relaxed) & bit) return VITCOP_OK;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e != cudaSuccess) return record_cuda(e);
    done.fetch_or(bit, std::memory_order_relaxed);
    return VITCOP_OK;
}

template <int BN, int MODE, int METRIC, bool SPATIAL>
int launch_one(const CUtensorMap& ma, const CUtensorMap& mb, const KernelArgs& k, cudaStream_t stream, bool pdl) {
    using S = GemmSmem<BN>;
    static std::atomic<unsigned long long> attr_done{0};
    auto kern = gram_tc_kernel<BN, MODE, METRIC, SPATIAL>;
    const int arc = allow_dynamic_smem(kern, S::kTotal, attr_done);
    if (arc != VITCOP_OK) return arc;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(k.total_tiles < num_sms() ? k.total_tiles : num_sms()));
    cfg.blockDim = dim3(gemm_threads(MODE));
    cfg.dynamicSmemBytes = S::kTotal;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_allowed(pdl) ? 1 : 0;
    KernelTimeScope timed(MODE == GRAM_RHO ? "gram_tc_kernel<rho>"
                          : MODE == GRAM_DELTA ? "gram_tc_kernel<delta>"
                          : MODE == GRAM_DIAG ? "gram_tc_kernel<diag>" : "gram_tc_kernel<sim>",
                          stream);
    return record_cuda(cudaLaunchKernelEx(&cfg, kern, ma, mb, k));
}

template <int BN>
int launch_bn(int mode, const CUtensorMap& ma, const CUtensorMap& mb, const KernelArgs& k, cudaStream_t stream,
              bool pdl) {
    const bool euclid = k.g.metric == 1;
    const bool spatial = k.g.tau2 >= 0.f && k.g.pos != nullptr;
    switch (mode) {
        case GRAM_RHO:
            return euclid ? launch_one<BN, GRAM_RHO, 1, false>(ma, mb, k, stream, pdl)
                          : launch_one<BN, GRAM_RHO, 0, false>(ma, mb, k, stream, pdl);
        case GRAM_DELTA:
            if (spatial)
                return euclid ? launch_one<BN, GRAM_DELTA, 1, true>(ma, mb, k, stream, pdl)
                              : launch_one<BN, GRAM_DELTA, 0, true>(ma, mb, k, stream, pdl);
            return euclid ? launch_one<BN, GRAM_DELTA, 1, false>(ma, mb, k, stream, pdl)
                          : launch_one<BN, GRAM_DELTA, 0, false>(ma, mb, k, stream, pdl);
        case GRAM_DIAG:
            if (BN != BM) return VITCOP_ERR_INVALID_ARG;
            return euclid ? launch_one<BM, GRAM_DIAG, 1, false>(ma, mb, k, stream, pdl)
                          : launch_one<BM, GRAM_DIAG, 0, false>(ma, mb, k, stream, pdl);
        default:
            return euclid ? launch_one<BN, GRAM_SIM, 1, false>(ma, mb, k, stream, pdl)
                          : launch_one<BN, GRAM_SIM, 0, false>(ma, mb, k, stream, pdl);
    }
}


template <int METRIC, bool SPATIAL>
int launch_resident_one(const CUtensorMap& ma, const CUtensorMap& mb, const KernelArgs& k, cudaStream_t stream) {
    using S = GemmSmem<kResidentBN>;
    static std::atomic<unsigned long long> attr_done{0};
    auto kern = gram_resident_kernel<METRIC, SPATIAL>;
    const int arc = allow_dynamic_smem(kern, S::kTotal, attr_done);
    if (arc != VITCOP_OK) return arc;
    const long long ctas = (k.total_tiles + kResidentUnits - 1) / kResidentUnits;
    cudaLaunchConfig_t cfg = {};
    // as many CTAs as there are SMs (never fewer than the units need): the shortest chain of units per CTA
    cfg.gridDim = dim3((unsigned)(k.total_tiles < num_sms() ? k.total_tiles : (ctas > num_sms() ? ctas : num_sms())));
    cfg.blockDim = dim3(64 + kResidentEpiThreads);
    cfg.dynamicSmemBytes = S::kTotal;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;          // all CTAs resident together: they wait for one another
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    KernelTimeScope timed("gram_resident_kernel", stream);
    return record_cuda(cudaLaunchKernelEx(&cfg, kern, ma, mb, k));
}

}  // namespace

int gram_num_sms() { return num_sms(); }

bool make_rowmajor_bf16_map(CUtensorMap* map, const void* base, int batches, int rows, int cols, int box_rows) {
    return make_feat_map(map, base, batches, rows, cols, box_rows);
}

unsigned long long gram_wait_limit_ns() { return g_wait_ns.load(); }

void gram_set_wait_debug(unsigned long long limit_ns, int expire_roles) {
    g_wait_ns.store(limit_ns ? limit_ns : kWaitLimitNs);
    g_expire_roles.store(expire_roles & 7);
}

bool gram_keeps_tiles(int B, int n) {
    return B > 0 && n >= kKeepTilesFromTokens && !gram_fits_resident(B, n) && gram_pick_bn(B, n) == 256;
}

int gram_pick_bn(int B, int n) {
    const long long ti = (n + BM - 1) / BM;
    const long long tiles128 = (long long)B * ti * (ti + 1) / 2;
    return tiles128 >= 4LL * num_sms() ? 256 : 128;
}

int launch_gram_sweep(int mode, const void* feat, const GramArgs& args, const GramTiling& tiling, cudaStream_t stream,
                      bool pdl) {
    KernelArgs k;
    k.g = args;
    k.t = tiling;
    if (mode == GRAM_SIM) {
        // plain rectangle: rows [row0, row_end) x all columns
        const int rows = args.row_end - args.row0;
        k.t.TI = (rows + BM - 1) / BM;
        k.t.TJ = (args.n + tiling.BN - 1) / tiling.BN;
        k.t.tiles_per_b = k.t.TI * k.t.TJ;
    } else {
        k.g.row0 = 0;
        k.g.row_end = args.n;
        if (mode == GRAM_DIAG) k.t.tiles_per_b = k.t.TI;        // one tile per 128-row block (tiling.BN == 128)
    }
    k.total_tiles = (long long)args.B * k.t.tiles_per_b;
    k.extra_units_per_b = 0;
    k.wait_ns = g_wait_ns.load();
    k.expire_roles = g_expire_roles.load();
    if (k.total_tiles <= 0) return VITCOP_OK;
    CUtensorMap ma, mb;
    if (!make_feat_map(&ma, feat, args.B, args.n, args.D, BM) ||
        !make_feat_map(&mb, feat, args.B, args.n, args.D, tiling.BN))
        return VITCOP_ERR_CUDA;
    return tiling.BN == 256 ? launch_bn<256>(mode, ma, mb, k, stream, pdl)
                            : launch_bn<128>(mode, ma, mb, k, stream, pdl);
}

bool gram_fits_resident(int B, int n) {
    static std::atomic<int> cooperative[kMaxDevices];     // the resident kernel needs a cooperative launch: 1 yes, 2 no
    const int dev = current_device();
    int c = cooperative[dev].load(std::memory_order_relaxed);
    if (c == 0) {
        int v = 0;
        c = (cudaDeviceGetAttribute(&v, cudaDevAttrCooperativeLaunch, dev) == cudaSuccess && v) ? 1 : 2;
        cooperative[dev].store(c, std::memory_order_relaxed);
    }
    if (c != 1) return false;
    const int ti = (n + BM - 1) / BM;
    const long long units = (long long)B * (ti + resident_extra_units(ti));
    return units > 0 && units <= (long long)kResidentUnits * num_sms();
}

bool gram_resident_takes_knorm(int H, int d) {
    // sixteen or more 16-byte pieces per row (the lane layout of the stand-alone kernel's widest variant), and at
    // least one chunk of eight tokens must fit the operand buffers
    if (H <= 0 || d <= 0 || d % 8 || d / 8 < 16) return false;
    return (long long)H * kKnChunkTokens * d * 2 <= (long long)GemmSmem<kResidentBN>::kTileBytes;
}

int launch_gram_resident(const void* feat, const GramArgs& args, const GramTiling& tiling, cudaStream_t stream) {
    KernelArgs k;
    k.g = args;
    k.t = tiling;
    k.g.row0 = 0;
    k.g.row_end = args.n;
    k.extra_units_per_b = resident_extra_units(k.t.TI);
    k.total_tiles = (long long)args.B * (k.t.TI + k.extra_units_per_b);
    k.wait_ns = g_wait_ns.load();
    k.expire_roles = g_expire_roles.load();
    if (k.total_tiles <= 0) return VITCOP_OK;
    if (tiling.BN != BM || k.total_tiles > (long long)kResidentUnits * num_sms()) return VITCOP_ERR_INVALID_ARG;
    CUtensorMap ma, mb;
    if (!make_feat_map(&ma, feat, args.B, args.n, args.D, BM) ||
        !make_feat_map(&mb, feat, args.B, args.n, args.D, kResidentBN))
        return VITCOP_ERR_CUDA;
    const bool euclid = args.metric == 1;
    const bool spatial = args.tau2 >= 0.f && args.pos != nullptr;
    if (spatial)
        return euclid ? launch_resident_one<1, true>(ma, mb, k, stream) : launch_resident_one<0, true>(ma, mb, k, stream);
    return euclid ? launch_resident_one<1, false>(ma, mb, k, stream) : launch_resident_one<0, false>(ma, mb, k, stream);
}

}  // namespace vitcop
