// Redundancy filter = Visual Information Clustering (Algorithm 2, Eq. 2 and Eq. 3) on one B200.
//
// Pipeline (all on one stream, no host synchronisation):
//   1. row_stats_kernel      |f_i|^2 in fp32 -> per-token weights (cosine: 1/|f_i|; euclid: |f_i|^2)
//   2. gram sweep, MODE_RHO  Gram tiles f_I . f_J^T on the tensor cores (tcgen05, fp32 accumulators in
//                            TMEM, operands staged by TMA); the epilogue turns each tile into squared
//                            distances, exp(-(d/d_c)^2) and per-row partial sums of Eq. 2
//   3. rho_reduce_kernel     fixed-order sum of the per-tile-column partials -> rho (deterministic)
//   4. gram sweep, MODE_DELTA the same tiles again; the epilogue keeps, per row, the nearest denser
//                            token inside the spatial radius (Eq. 3) as a packed (d^2, j) 64-bit minimum
//   5. vic_finalize_kernel   gamma = rho * delta, radix-select of the centres, pointer jumping over the
//                            parent forest, orphan fallback, labels (Algorithm 2, steps 3-4)
// The Gram matrix is never written to memory: it is recomputed for the second sweep.
//
// The Gram is taken on the RAW bf16 features (bf16 x bf16 products are exact in fp32); the L2
// normalisation enters as fp32 factors in the epilogue, so the similarity keeps fp32 accuracy.
#include <cuda.h>

#include <cstdlib>
#include <cstring>

#include "internal.cuh"

namespace vitcop {
namespace {

// ------------------------------------------------------------------------------------------------
// constants
// ------------------------------------------------------------------------------------------------
constexpr int BM = 128;            // tile rows  (UMMA M)
constexpr int BK = 64;             // k-block: 64 bf16 = 128 bytes = one 128B-swizzle row
constexpr int UMMA_K = 16;
constexpr int kGemmThreads = 192;  // warp 0: TMA producer, warp 1: MMA issuer + TMEM owner, warps 2-5: epilogue
constexpr int kEpiThreads = 128;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // bounded waits: after 2 s give up, flag VITCOP_ERR_TIMEOUT and leave
constexpr unsigned long long kDrainLimitNs = 20000000ull;    // bounded waits for this CTA's own copies / MMAs after giving up

enum { MODE_RHO = 0, MODE_DELTA = 1, MODE_SIM = 2 };

struct GemmArgs {
    int B, n, D;
    int row0, row_end;          // rows [row0, row_end) are produced (the filter uses [0, n))
    int TI, TJ;                 // tile counts along rows / columns
    int metric;
    float neg_c_log2e;          // -(log2 e) / d_c^2
    float tau2;                 // tau^2, < 0: no spatial test
    const float* w;             // [B, n] per-token factor multiplying the Gram value (cosine 1/|f|, euclid 1)
    const float* a;             // [B, n] additive term (cosine 1, euclid |f|^2):  d^2 = a_i + a_j - 2 g w_i w_j
    const float* rho;           // [B, n]                 (MODE_DELTA)
    const float* pos;           // [B, n, 2] or nullptr   (MODE_DELTA)
    float* rho_part;            // [B, TJ, n_pad]         (MODE_RHO)
    int n_pad;
    unsigned long long* best;   // [B, n] packed (d2 bits << 32 | j), ~0 = none   (MODE_DELTA)
    float* sim_out;             // [B, row_end-row0, n]   (MODE_SIM)
    int* status;
};

// ------------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    return done != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait.  Returns false (after raising `abort_flag`) when the time limit is hit or another role gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    for (uint32_t it = 1;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 0u) {
            if (*abort_flag) return false;
            if (global_ns() - t0 > kWaitLimitNs) break;
        }
    }
    *abort_flag = 1;
    return false;
}
// Bounded wait without side effects, used while leaving after a timeout.
__device__ __forceinline__ void mbar_drain(uint32_t bar, uint32_t parity) {
    const unsigned long long t0 = global_ns();
    while (!mbar_try_wait(bar, parity))
        if (global_ns() - t0 > kDrainLimitNs) break;
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1,
                                            int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, bf16 inputs, fp32 accumulate; issued by one thread.
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// 32 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int u = 0; u < 32; ++u) v[u] = __uint_as_float(r[u]);
}
__device__ __forceinline__ void epi_bar_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
// Barrier over the 128 epilogue threads that also ORs a predicate: every thread gets the same answer.
__device__ __forceinline__ bool epi_bar_or(bool pred) {
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 p, %1, 0;\n\t"
        "bar.red.or.pred q, 1, 128, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(out)
        : "r"((uint32_t)pred)
        : "memory");
    return out != 0;
}

// Shared-memory matrix descriptor of a K-major bf16 tile whose rows are 128 bytes (64 elements) wide,
// laid out by TMA with the 128-byte swizzle: 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc_k128(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr >> 4) & 0x3FFFu);          // start address
    d |= (uint64_t)0 << 16;                               // leading byte offset: unused for this layout
    d |= (uint64_t)((1024u >> 4) & 0x3FFFu) << 32;        // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                               // descriptor version (sm_100)
    d |= (uint64_t)2 << 61;                               // swizzle mode: 128 bytes
    return d;
}
// Instruction descriptor: D fp32, A and B bf16, both K-major, M = 128, N = BN.
__host__ __device__ constexpr uint32_t umma_idesc_bf16(int M, int N) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// ------------------------------------------------------------------------------------------------
// Epilogue arithmetic shared by the tensor-core engine and the diagnostic SIMT engine
// ------------------------------------------------------------------------------------------------
struct RowState {
    // row-side constants
    int i;                 // global token index of this thread's row
    float w_i, a_i, rho_i, x_i, y_i;
    // accumulators
    float acc;             // MODE_RHO
    float best;            // MODE_DELTA
    int best_j;
};

struct ColArrays {          // per tile column data in shared memory
    float *w, *a, *rho, *x, *y;
};

template <int MODE>
__device__ __forceinline__ void epi_process_chunk(const GemmArgs& g, RowState& rs, const ColArrays& col,
                                                  const float (&v)[32], int jl0 /*tile-local first column*/, int J0,
                                                  int b, bool row_valid) {
    const int n = g.n;
    if (MODE == MODE_SIM) {
        if (!row_valid) return;
        float* o = g.sim_out + ((size_t)b * (g.row_end - g.row0) + (rs.i - g.row0)) * n;
#pragma unroll
        for (int u = 0; u < 32; ++u) {
            const int j = J0 + jl0 + u;
            if (j < n) o[j] = g.metric == 0 ? (v[u] * rs.w_i) * col.w[jl0 + u] : v[u];
        }
        return;
    }
    const bool full = (J0 + jl0 + 32 <= n);
    const bool has_diag = (rs.i >= J0 + jl0) && (rs.i < J0 + jl0 + 32);
    if (MODE == MODE_RHO) {
        float acc = rs.acc;
        if (full && !__any_sync(0xffffffffu, has_diag)) {
#pragma unroll
            for (int u = 0; u < 32; ++u) {
                const float x = (v[u] * rs.w_i) * col.w[jl0 + u];
                const float d2 = fmaxf(0.f, fmaf(-2.f, x, rs.a_i + col.a[jl0 + u]));
                acc += exp2f(d2 * g.neg_c_log2e);
            }
        } else {
#pragma unroll
            for (int u = 0; u < 32; ++u) {
                const int j = J0 + jl0 + u;
                const float x = (v[u] * rs.w_i) * col.w[jl0 + u];
                const float d2 = fmaxf(0.f, fmaf(-2.f, x, rs.a_i + col.a[jl0 + u]));
                const float e = exp2f(d2 * g.neg_c_log2e);
                if (j < n && j != rs.i) acc += e;
            }
        }
        rs.acc = acc;
    } else {  // MODE_DELTA
        const bool spatial = g.tau2 >= 0.f && g.pos != nullptr;
#pragma unroll
        for (int u = 0; u < 32; ++u) {
            const float x = (v[u] * rs.w_i) * col.w[jl0 + u];
            const float d2 = fmaxf(0.f, fmaf(-2.f, x, rs.a_i + col.a[jl0 + u]));
            if (d2 < rs.best) {
                const int j = J0 + jl0 + u;
                const float rj = col.rho[jl0 + u];
                bool ok = j < n && j != rs.i && (rj > rs.rho_i || (rj == rs.rho_i && j < rs.i));
                if (ok && spatial) {
                    const float dx = col.x[jl0 + u] - rs.x_i, dy = col.y[jl0 + u] - rs.y_i;
                    ok = fmaf(dx, dx, dy * dy) <= g.tau2;
                }
                if (ok) {
                    rs.best = d2;
                    rs.best_j = j;
                }
            }
        }
    }
}

template <int MODE>
__device__ __forceinline__ void epi_load_cols(const GemmArgs& g, const ColArrays& col, int b, int J0, int BN, int e) {
    for (int jl = e; jl < BN; jl += kEpiThreads) {
        const int j = J0 + jl;
        const bool ok = j < g.n;
        const size_t o = (size_t)b * g.n + j;
        col.w[jl] = ok ? g.w[o] : 0.f;
        col.a[jl] = ok ? g.a[o] : 0.f;
        if (MODE == MODE_DELTA) {
            col.rho[jl] = ok ? g.rho[o] : 0.f;
            col.x[jl] = (ok && g.pos) ? g.pos[2 * o] : 0.f;
            col.y[jl] = (ok && g.pos) ? g.pos[2 * o + 1] : 0.f;
        }
    }
}

template <int MODE>
__device__ __forceinline__ void epi_row_begin(const GemmArgs& g, RowState& rs, int b, int i, bool row_valid) {
    rs.i = i;
    const size_t o = (size_t)b * g.n + i;
    rs.w_i = row_valid ? g.w[o] : 0.f;
    rs.a_i = row_valid ? g.a[o] : 0.f;
    rs.acc = 0.f;
    rs.best = __int_as_float(0x7f800000);
    rs.best_j = -1;
    rs.rho_i = 0.f; rs.x_i = 0.f; rs.y_i = 0.f;
    if (MODE == MODE_DELTA && row_valid) {
        rs.rho_i = g.rho[o];
        if (g.pos) { rs.x_i = g.pos[2 * o]; rs.y_i = g.pos[2 * o + 1]; }
    }
}

template <int MODE>
__device__ __forceinline__ void epi_row_end(const GemmArgs& g, const RowState& rs, int b, int tj, bool row_valid) {
    if (!row_valid) return;
    if (MODE == MODE_RHO) {
        g.rho_part[((size_t)b * g.TJ + tj) * g.n_pad + rs.i] = rs.acc;
    } else if (MODE == MODE_DELTA) {
        if (rs.best_j >= 0) {
            const unsigned long long packed =
                ((unsigned long long)__float_as_uint(rs.best) << 32) | (unsigned long long)(uint32_t)rs.best_j;
            atomicMin(g.best + (size_t)b * g.n + rs.i, packed);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Tensor-core Gram sweep: persistent, warp-specialised, one CTA per SM.
//   smem per stage: A tile [128 rows][64 k] + B tile [BN rows][64 k], both 128B-swizzled by TMA
//   TMEM: two fp32 accumulators of BN columns (double-buffered against the epilogue)
// ------------------------------------------------------------------------------------------------
template <int BN>
struct GemmSmem {
    static constexpr int kStages = (BN == 128) ? 6 : 4;
    static constexpr int kABytes = BM * BK * 2;
    static constexpr int kBBytes = BN * BK * 2;
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kTileBytes = kStages * kStageBytes;
    static constexpr int kColBytes = 5 * BN * 4;
    static constexpr int kBarBytes = 256;
    static constexpr int kTotal = 1024 /*alignment slack*/ + kTileBytes + kColBytes + kBarBytes;
};

template <int BN, int MODE>
__global__ void __launch_bounds__(kGemmThreads, 1)
gram_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const GemmArgs g) {
    using S = GemmSmem<BN>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;                 // 1024-byte aligned for the 128B swizzle
    uint8_t* gen = smem_raw + (tiles - raw);
    float* colbase = reinterpret_cast<float*>(gen + S::kTileBytes);
    uint64_t* bars = reinterpret_cast<uint64_t*>(gen + S::kTileBytes + S::kColBytes);
    // barriers: full[kStages], empty[kStages], tmem_full[2], tmem_empty[2], drain
    const uint32_t bar_full = smem_u32(bars);
    const uint32_t bar_empty = bar_full + 8 * S::kStages;
    const uint32_t bar_tfull = bar_empty + 8 * S::kStages;
    const uint32_t bar_tempty = bar_tfull + 16;
    const uint32_t bar_drain = bar_tempty + 16;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * S::kStages + 5);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr uint32_t kTmemCols = 2 * BN;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S::kStages; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(bar_tfull + 8 * a, 1);
            mbar_init(bar_tempty + 8 * a, kEpiThreads);
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

    grid_dependency_wait();   // inputs written by the preceding kernel on the stream (PDL)

    const int tiles_per_b = g.TI * g.TJ;
    const long long total_tiles = (long long)g.B * tiles_per_b;
    const int KB = g.D / BK;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            uint32_t issued = 0, issued_parity = 0;        // per stage: a load was issued / parity of its phase
            bool ok = true;
            for (long long t = blockIdx.x; ok && t < total_tiles; t += gridDim.x) {
                const int b = (int)(t / tiles_per_b);
                const int r = (int)(t - (long long)b * tiles_per_b);
                const int ti = r / g.TJ, tj = r - ti * g.TJ;
                const int I0 = g.row0 + ti * BM, J0 = tj * BN;
                for (int kb = 0; kb < KB; ++kb) {
                    if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t sa = tiles + stage * S::kStageBytes;
                    mbar_expect_tx(bar_full + 8 * stage, S::kStageBytes);
                    tma_load_3d(sa, &map_a, bar_full + 8 * stage, kb * BK, I0, b);
                    tma_load_3d(sa + S::kABytes, &map_b, bar_full + 8 * stage, kb * BK, J0, b);
                    issued |= 1u << stage;
                    issued_parity = (issued_parity & ~(1u << stage)) | (phase << stage);
                    if (++stage == S::kStages) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok) {
                // leaving early: give the copies still in flight into this CTA's shared memory time to land
                for (int s = 0; s < S::kStages; ++s)
                    if (issued >> s & 1u) mbar_drain(bar_full + 8 * s, issued_parity >> s & 1u);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(BM, BN);
            uint32_t stage = 0, phase = 0;
            uint32_t acc = 0, acc_phase = 0;
            bool ok = true;
            for (long long t = blockIdx.x; ok && t < total_tiles; t += gridDim.x) {
                if (!mbar_wait(bar_tempty + 8 * acc, acc_phase ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * BN;
                for (int kb = 0; kb < KB; ++kb) {
                    if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = tiles + stage * S::kStageBytes;
                    const uint64_t da = umma_desc_k128(sa), db = umma_desc_k128(sa + S::kABytes);
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k) {
                        // advancing 16 elements (32 bytes) along K inside the swizzle row: +2 in address units
                        tc_mma_bf16(d_tmem, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc,
                                    (kb > 0 || k > 0) ? 1u : 0u);
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
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        const int e = threadIdx.x - 64;                    // 0..127
        const int quarter = warp & 3;                      // TMEM lane quarter this warp may read
        const int rl = quarter * 32 + lane;                // tile-local row == TMEM lane
        ColArrays col;
        col.w = colbase; col.a = colbase + BN; col.rho = colbase + 2 * BN; col.x = colbase + 3 * BN;
        col.y = colbase + 4 * BN;
        uint32_t acc = 0, acc_phase = 0;
        bool ok = true;
        for (long long t = blockIdx.x; t < total_tiles; t += gridDim.x) {
            const int b = (int)(t / tiles_per_b);
            const int r = (int)(t - (long long)b * tiles_per_b);
            const int ti = r / g.TJ, tj = r - ti * g.TJ;
            const int I0 = g.row0 + ti * BM, J0 = tj * BN;
            const int i = I0 + rl;
            const bool row_valid = i < g.row_end;
            epi_load_cols<MODE>(g, col, b, J0, BN, e);
            RowState rs;
            epi_row_begin<MODE>(g, rs, b, i, row_valid);
            epi_bar_sync();
            if (ok) ok = mbar_wait(bar_tfull + 8 * acc, acc_phase, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (ok) {
                tc_fence_after();
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * BN;
#pragma unroll 1
                for (int c = 0; c < BN / 32; ++c) {
                    float v[32];
                    tmem_ld32(taddr + c * 32, v);
                    epi_process_chunk<MODE>(g, rs, col, v, c * 32, J0, b, row_valid);
                }
                tc_fence_before();
                mbar_arrive(bar_tempty + 8 * acc);
                epi_row_end<MODE>(g, rs, b, tj, row_valid);
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
            // column arrays are rewritten for the next tile; all four warps leave together or not at all
            if (epi_bar_or(!ok)) break;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
    if (threadIdx.x == 0 && *abort_flag && g.status) atomicMax(g.status, VITCOP_ERR_TIMEOUT);
    grid_dependency_launch_dependents();
}

// ------------------------------------------------------------------------------------------------
// Diagnostic SIMT engine (environment VITCOP_GRAM_ENGINE=simt): same tiles and the same epilogue, Gram
// values from plain fp32 FMAs.  One CTA of 128 threads per (128 x 32) tile piece; slow by design.
// ------------------------------------------------------------------------------------------------
template <int MODE>
__global__ void __launch_bounds__(kEpiThreads)
gram_simt_kernel(const uint16_t* __restrict__ feat, const GemmArgs g) {
    constexpr int BN = 128, CH = 32;
    __shared__ float fj[CH][BK + 1];
    __shared__ float colbuf[5 * BN];
    const int b = blockIdx.z;
    const int I0 = g.row0 + blockIdx.y * BM, J0 = blockIdx.x * BN;
    const int e = threadIdx.x;
    const int i = I0 + e;
    const bool row_valid = i < g.row_end;
    ColArrays col;
    col.w = colbuf; col.a = colbuf + BN; col.rho = colbuf + 2 * BN; col.x = colbuf + 3 * BN; col.y = colbuf + 4 * BN;
    epi_load_cols<MODE>(g, col, b, J0, BN, e);
    RowState rs;
    epi_row_begin<MODE>(g, rs, b, i, row_valid);
    const uint16_t* fi = feat + ((size_t)b * g.n + (row_valid ? i : 0)) * g.D;
    for (int c = 0; c < BN / CH; ++c) {
        float v[32];
#pragma unroll
        for (int u = 0; u < 32; ++u) v[u] = 0.f;
        for (int k0 = 0; k0 < g.D; k0 += BK) {
            __syncthreads();
            for (int q = e; q < CH * BK; q += kEpiThreads) {
                const int jj = q / BK, kk = q - jj * BK;
                const int j = J0 + c * CH + jj;
                fj[jj][kk] =
                    j < g.n ? __uint_as_float((uint32_t)feat[((size_t)b * g.n + j) * g.D + k0 + kk] << 16) : 0.f;
            }
            __syncthreads();
            for (int kk = 0; kk < BK; ++kk) {
                const float a = row_valid ? __uint_as_float((uint32_t)fi[k0 + kk] << 16) : 0.f;
#pragma unroll
                for (int u = 0; u < 32; ++u) v[u] = fmaf(a, fj[u][kk], v[u]);
            }
        }
        epi_process_chunk<MODE>(g, rs, col, v, c * CH, J0, b, row_valid);
    }
    epi_row_end<MODE>(g, rs, b, blockIdx.x, row_valid);
}

// ------------------------------------------------------------------------------------------------
// small kernels
// ------------------------------------------------------------------------------------------------
// One warp per token: |f|^2 in fp32, then the epilogue factors.  Also resets the packed minima.
__global__ void row_stats_kernel(const uint4* __restrict__ feat, int total_rows, int D8, int metric,
                                 float* __restrict__ w, float* __restrict__ a, unsigned long long* __restrict__ best) {
    grid_dependency_wait();
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= total_rows) return;
    const uint4* p = feat + (size_t)row * D8;
    float s0 = 0.f, s1 = 0.f;
    for (int c = lane; c < D8; c += 32) {
        const uint4 v = p[c];
        float x;
        x = bf16lo(v.x); s0 = fmaf(x, x, s0);  x = bf16hi(v.x); s1 = fmaf(x, x, s1);
        x = bf16lo(v.y); s0 = fmaf(x, x, s0);  x = bf16hi(v.y); s1 = fmaf(x, x, s1);
        x = bf16lo(v.z); s0 = fmaf(x, x, s0);  x = bf16hi(v.z); s1 = fmaf(x, x, s1);
        x = bf16lo(v.w); s0 = fmaf(x, x, s0);  x = bf16hi(v.w); s1 = fmaf(x, x, s1);
    }
    float s = s0 + s1;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
    if (lane == 0) {
        if (metric == 0) {
            w[row] = s > 0.f ? 1.0f / sqrtf(s) : 0.f;
            a[row] = 1.f;
        } else {
            w[row] = 1.f;
            a[row] = s;
        }
        if (best) best[row] = ~0ull;
    }
    grid_dependency_launch_dependents();
}

// rho[b,i] = sum over tile columns, in tile order (fixed order => reproducible bits).
__global__ void rho_reduce_kernel(const float* __restrict__ part, int B, int n, int TJ, int n_pad,
                                  float* __restrict__ rho, float* __restrict__ rho_user) {
    grid_dependency_wait();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    const int b = blockIdx.y;
    if (i < n) {
        float s = 0.f;
        for (int t = 0; t < TJ; ++t) s += part[((size_t)b * TJ + t) * n_pad + i];
        rho[(size_t)b * n + i] = s;
        if (rho_user) rho_user[(size_t)b * n + i] = s;
    }
    grid_dependency_launch_dependents();
}

// ------------------------------------------------------------------------------------------------
// Centres, forest roots and labels: one CTA per sample.
// ------------------------------------------------------------------------------------------------
constexpr int kFinThreads = 1024;

__device__ __forceinline__ uint32_t fin_prefix_count(bool flag, uint32_t* warp_sums, uint32_t& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t bal = __ballot_sync(0xffffffffu, flag);
    const uint32_t before = __popc(bal & ((1u << lane) - 1u));
    if (lane == 0) warp_sums[warp] = __popc(bal);
    __syncthreads();
    uint32_t v = warp_sums[lane];
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, v, off);
        if (lane >= off) v += t;
    }
    total = __shfl_sync(0xffffffffu, v, 31);
    const uint32_t base = __shfl_sync(0xffffffffu, v, (warp + 31) & 31);
    __syncthreads();
    return (warp == 0 ? 0u : base) + before;
}

// Shared memory: keys[n] (uint64; later reused as next[n] int32), isc[n] (uint8), centres[nc] (int32).
__global__ void __launch_bounds__(kFinThreads)
vic_finalize_kernel(const uint16_t* __restrict__ feat, int n, int D, int n_centers, const float* __restrict__ rho,
                    const unsigned long long* __restrict__ best, const float* __restrict__ w,
                    const float* __restrict__ a, int32_t* __restrict__ label, int32_t* __restrict__ n_clusters,
                    float* __restrict__ delta2_user, int32_t* __restrict__ parent_user) {
    extern __shared__ __align__(16) uint8_t fin_smem[];
    unsigned long long* keys = reinterpret_cast<unsigned long long*>(fin_smem);
    int32_t* nxt = reinterpret_cast<int32_t*>(fin_smem);              // aliases keys after the selection
    uint8_t* isc = fin_smem + (size_t)n * 8;
    int32_t* centres = reinterpret_cast<int32_t*>(fin_smem + (size_t)n * 8 + (((size_t)n + 15) & ~(size_t)15));
    __shared__ uint32_t hist[256];
    __shared__ uint32_t warp_sums[32];
    __shared__ uint32_t s_digit, s_krem;

    grid_dependency_wait();
    const int b = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    rho += (size_t)b * n;
    best += (size_t)b * n;
    w += (size_t)b * n;
    a += (size_t)b * n;
    label += (size_t)b * n;
    feat += (size_t)b * n * D;
    if (delta2_user) delta2_user += (size_t)b * n;
    if (parent_user) parent_user += (size_t)b * n;
    const int nc = min(n_centers, n);

    // rank key, ascending = better centre candidate: ~( orphan ? (0xFFFFFFFF, rho) : (gamma, rho) )
    for (int i = tid; i < n; i += kFinThreads) {
        const unsigned long long p = best[i];
        const bool orphan = p == ~0ull;
        const float d2 = orphan ? __int_as_float(0x7f800000) : __uint_as_float((uint32_t)(p >> 32));
        const int par = orphan ? -1 : (int)(uint32_t)(p & 0xFFFFFFFFull);
        if (delta2_user) delta2_user[i] = d2;
        if (parent_user) parent_user[i] = par;
        const float r = rho[i];
        const uint32_t hi = orphan ? 0xFFFFFFFFu : __float_as_uint(r * sqrtf(d2));
        keys[i] = ~(((unsigned long long)hi << 32) | (unsigned long long)__float_as_uint(r));
    }
    __syncthreads();

    // ---- radix select of the nc smallest keys (8 passes of 8 bits), ties -> lower index
    unsigned long long T = ~0ull;
    uint32_t krem = 0;
    if (nc > 0 && nc < n) {
        unsigned long long prefix = 0;
        krem = (uint32_t)nc;
        for (int pass = 0; pass < 8; ++pass) {
            const int shift = 56 - 8 * pass;
            const unsigned long long hi_mask = pass == 0 ? 0ull : (~0ull << (shift + 8));
            if (tid < 256) hist[tid] = 0;
            __syncthreads();
            for (int base = 0; base < n; base += kFinThreads) {
                const int i = base + tid;
                int dig = -1;
                if (i < n) {
                    const unsigned long long key = keys[i];
                    if ((key & hi_mask) == prefix) dig = (int)((key >> shift) & 255ull);
                }
                const uint32_t peers = __match_any_sync(0xffffffffu, dig);
                if (dig >= 0 && lane == __ffs(peers) - 1) atomicAdd(&hist[dig], (uint32_t)__popc(peers));
            }
            __syncthreads();
            const uint32_t c = tid < 256 ? hist[tid] : 0u;
            uint32_t v = c;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const uint32_t t = __shfl_up_sync(0xffffffffu, v, off);
                if (lane >= off) v += t;
            }
            if (lane == 31) warp_sums[warp] = v;
            __syncthreads();
            if (tid < 256) {
                uint32_t basew = 0;
                for (int q = 0; q < warp; ++q) basew += warp_sums[q];
                const uint32_t incl = basew + v, excl = incl - c;
                if (excl < krem && krem <= incl) {
                    s_digit = (uint32_t)tid;
                    s_krem = krem - excl;
                }
            }
            __syncthreads();
            prefix |= (unsigned long long)s_digit << shift;
            krem = s_krem;
            __syncthreads();
        }
        T = prefix;
    }
    // ---- centre flags + ascending centre list
    {
        uint32_t eq_running = 0, c_running = 0;
        for (int base = 0; base < n; base += kFinThreads) {
            const int i = base + tid;
            const unsigned long long key = i < n ? keys[i] : ~0ull;
            bool f;
            if (nc <= 0) f = false;
            else if (nc >= n) f = i < n;
            else {
                const bool eq = i < n && key == T;
                uint32_t eq_total;
                const uint32_t eq_rank = eq_running + fin_prefix_count(eq, warp_sums, eq_total);
                eq_running += eq_total;
                f = i < n && (key < T || (eq && eq_rank < krem));
            }
            uint32_t c_total;
            const uint32_t r = c_running + fin_prefix_count(f, warp_sums, c_total);
            c_running += c_total;
            if (i < n) isc[i] = f ? 1 : 0;
            if (f && r < (uint32_t)nc) centres[r] = i;
        }
    }
    __syncthreads();   // keys are dead from here on; nxt aliases them

    // ---- forest roots by pointer jumping: a centre or an orphan is its own root
    for (int i = tid; i < n; i += kFinThreads) {
        const unsigned long long p = best[i];
        const int par = (p == ~0ull) ? -1 : (int)(uint32_t)(p & 0xFFFFFFFFull);
        nxt[i] = (isc[i] || par < 0 || par >= n) ? i : par;
    }
    __syncthreads();
    for (int round = 0; round < 16; ++round) {
        int changed = 0;
        for (int i = tid; i < n; i += kFinThreads) {
            const int p = nxt[i];
            const int q = nxt[p];
            if (q != p) {
                nxt[i] = q;       // any value read here is an ancestor of i, roots are fixed points
                changed = 1;
            }
        }
        if (!__syncthreads_or(changed)) break;
    }

    // ---- labels; a root that is an orphan but not a centre joins the nearest centre (feature distance)
    for (int i = tid; i < n; i += kFinThreads) {
        const int root = nxt[i];
        label[i] = isc[root] ? root : -1 - root;
    }
    __syncthreads();
    if (nc > 0) {
        for (int o = warp; o < n; o += kFinThreads / 32) {
            if (isc[o] || nxt[o] != o) continue;                   // only surplus orphans (warp-uniform)
            const uint16_t* fo = feat + (size_t)o * D;
            float bestd = __int_as_float(0x7f800000);
            int bestc = centres[0];
            for (int q = 0; q < nc; ++q) {
                const int c = centres[q];
                const uint16_t* fc = feat + (size_t)c * D;
                float dot = 0.f;
                for (int k = lane * 2; k < D; k += 64) {
                    const uint32_t u = *reinterpret_cast<const uint32_t*>(fo + k);
                    const uint32_t v = *reinterpret_cast<const uint32_t*>(fc + k);
                    dot = fmaf(bf16lo(u), bf16lo(v), dot);
                    dot = fmaf(bf16hi(u), bf16hi(v), dot);
                }
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
                const float d2 = fmaxf(0.f, fmaf(-2.f, (dot * w[o]) * w[c], a[o] + a[c]));
                if (d2 < bestd) { bestd = d2; bestc = c; }
            }
            if (lane == 0) nxt[o] = -1 - bestc;                      // remember the adopted centre at the root
        }
    }
    __syncthreads();
    for (int i = tid; i < n; i += kFinThreads) {
        const int l = label[i];
        if (l < 0) {
            const int root = -1 - l;
            const int adopted = nxt[root];
            label[i] = adopted < 0 ? -1 - adopted : root;
        }
    }
    if (tid == 0) n_clusters[b] = nc;
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

bool use_simt_engine() {
    const char* e = std::getenv("VITCOP_GRAM_ENGINE");
    return e && std::strcmp(e, "simt") == 0;
}

int num_sms() {
    static int sms = 0;
    if (!sms) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return 148;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) sms = 148;
    }
    return sms;
}

template <int BN, int MODE>
int launch_gram_tc(const CUtensorMap& ma, const CUtensorMap& mb, const GemmArgs& g, cudaStream_t stream, bool pdl) {
    using S = GemmSmem<BN>;
    static bool attr_done = false;
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(gram_tc_kernel<BN, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             S::kTotal);
        if (e != cudaSuccess) return record_cuda(e);
        attr_done = true;
    }
    const long long total = (long long)g.B * g.TI * g.TJ;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(total < num_sms() ? total : num_sms()));
    cfg.blockDim = dim3(kGemmThreads);
    cfg.dynamicSmemBytes = S::kTotal;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_allowed(pdl) ? 1 : 0;
    KernelTimeScope timed(MODE == MODE_RHO ? "gram_tc_kernel<rho>" : MODE == MODE_DELTA ? "gram_tc_kernel<delta>" : "gram_tc_kernel<sim>", stream);
    return record_cuda(cudaLaunchKernelEx(&cfg, gram_tc_kernel<BN, MODE>, ma, mb, g));
}

template <int MODE>
int launch_gram(const void* feat, GemmArgs g, cudaStream_t stream, bool pdl, int* tj_used) {
    const int rows = g.row_end - g.row0;
    g.TI = (rows + BM - 1) / BM;
    if (use_simt_engine()) {
        g.TJ = (g.n + 127) / 128;
        if (tj_used) *tj_used = g.TJ;
        dim3 grid(g.TJ, g.TI, g.B);
        KernelTimeScope timed("gram_simt_kernel", stream);
        gram_simt_kernel<MODE><<<grid, kEpiThreads, 0, stream>>>(static_cast<const uint16_t*>(feat), g);
        return record_cuda(cudaGetLastError());
    }
    // wide tiles halve the operand traffic per flop; narrow tiles fill the SMs when the problem is small
    const long long tiles128 = (long long)g.B * g.TI * ((g.n + 127) / 128);
    const bool wide = tiles128 >= 4LL * num_sms();
    const int BN = wide ? 256 : 128;
    g.TJ = (g.n + BN - 1) / BN;
    if (tj_used) *tj_used = g.TJ;
    CUtensorMap ma, mb;
    if (!make_feat_map(&ma, feat, g.B, g.n, g.D, BM) || !make_feat_map(&mb, feat, g.B, g.n, g.D, BN))
        return VITCOP_ERR_CUDA;
    return wide ? launch_gram_tc<256, MODE>(ma, mb, g, stream, pdl) : launch_gram_tc<128, MODE>(ma, mb, g, stream, pdl);
}

// Workspace of the filter: status | w | a | rho | best | rho partials [B, ceil(n/128), n_pad]
struct FilterWs {
    size_t off_w, off_a, off_rho, off_best, off_part, total;
    int n_pad;
    FilterWs(int B, int n) {
        n_pad = (n + BM - 1) / BM * BM;
        size_t o = kStatusBytes;
        const size_t bn = (size_t)B * n;
        off_w = o;    o += align_up(bn * 4, 256);
        off_a = o;    o += align_up(bn * 4, 256);
        off_rho = o;  o += align_up(bn * 4, 256);
        off_best = o; o += align_up(bn * 8, 256);
        off_part = o; o += align_up((size_t)B * ((n + 127) / 128) * n_pad * 4, 256);
        total = o;
    }
};

}  // namespace

size_t filter_workspace_bytes(int B, int n, int D) {
    (void)D;
    return FilterWs(B, n).total;
}
size_t similarity_workspace_bytes(int B, int n, int D) {
    (void)D;
    return kStatusBytes + 2 * align_up((size_t)B * n * 4, 256);
}

int launch_filter(const void* feat, const float* pos, int B, int n, int D, const vitcop_filter_params& p,
                  int n_centers, int32_t* label, int32_t* n_clusters, float* rho_user, float* delta2_user,
                  int32_t* parent_user, void* workspace, cudaStream_t stream) {
    FilterWs l(B, n);
    char* ws = static_cast<char*>(workspace);
    float* w = reinterpret_cast<float*>(ws + l.off_w);
    float* a = reinterpret_cast<float*>(ws + l.off_a);
    float* rho = reinterpret_cast<float*>(ws + l.off_rho);
    unsigned long long* best = reinterpret_cast<unsigned long long*>(ws + l.off_best);
    float* part = reinterpret_cast<float*>(ws + l.off_part);

    const int rows = B * n;
    int rc;
    {
        KernelTimeScope timed("row_stats_kernel", stream);
        row_stats_kernel<<<(rows + 7) / 8, 256, 0, stream>>>(static_cast<const uint4*>(feat), rows, D / 8, p.metric, w,
                                                             a, best);
        rc = record_cuda(cudaGetLastError());
    }
    if (rc != VITCOP_OK) return rc;

    GemmArgs g = {};
    g.B = B; g.n = n; g.D = D; g.row0 = 0; g.row_end = n; g.metric = p.metric;
    g.neg_c_log2e = -1.4426950408889634f / (p.d_c * p.d_c);
    g.tau2 = (p.tau >= 0.f && pos) ? p.tau * p.tau : -1.f;
    g.w = w; g.a = a; g.rho = rho; g.pos = pos; g.rho_part = part; g.n_pad = l.n_pad; g.best = best;
    g.sim_out = nullptr; g.status = reinterpret_cast<int*>(ws);

    int TJ = 0;
    rc = launch_gram<MODE_RHO>(feat, g, stream, true, &TJ);
    if (rc != VITCOP_OK) return rc;
    {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((n + 255) / 256, B);
        cfg.blockDim = dim3(256);
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = pdl_allowed(true) ? 1 : 0;
        KernelTimeScope timed("rho_reduce_kernel", stream);
        rc = record_cuda(cudaLaunchKernelEx(&cfg, rho_reduce_kernel, (const float*)part, B, n, TJ, l.n_pad, rho,
                                            rho_user));
        if (rc != VITCOP_OK) return rc;
    }
    rc = launch_gram<MODE_DELTA>(feat, g, stream, true, nullptr);
    if (rc != VITCOP_OK) return rc;

    const int nc = n_centers < n ? n_centers : n;
    const size_t smem = (size_t)n * 8 + (((size_t)n + 15) & ~(size_t)15) + (size_t)(nc > 0 ? nc : 1) * 4 + 16;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(vic_finalize_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return record_cuda(e);
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(B);
    cfg.blockDim = dim3(kFinThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_allowed(true) ? 1 : 0;
    KernelTimeScope timed("vic_finalize_kernel", stream);
    return record_cuda(cudaLaunchKernelEx(&cfg, vic_finalize_kernel, static_cast<const uint16_t*>(feat), n, D, nc,
                                          (const float*)rho, (const unsigned long long*)best, (const float*)w,
                                          (const float*)a, label, n_clusters, delta2_user, parent_user));
}

int launch_similarity_rows(const void* feat, int B, int n, int D, int metric, int row_begin, int row_end, float* out,
                           void* workspace, cudaStream_t stream) {
    char* ws = static_cast<char*>(workspace);
    float* w = reinterpret_cast<float*>(ws + kStatusBytes);
    float* a = reinterpret_cast<float*>(ws + kStatusBytes + align_up((size_t)B * n * 4, 256));
    const int rows = B * n;
    int rc;
    {
        KernelTimeScope timed("row_stats_kernel", stream);
        row_stats_kernel<<<(rows + 7) / 8, 256, 0, stream>>>(static_cast<const uint4*>(feat), rows, D / 8, metric, w, a,
                                                             nullptr);
        rc = record_cuda(cudaGetLastError());
    }
    if (rc != VITCOP_OK) return rc;
    GemmArgs g = {};
    g.B = B; g.n = n; g.D = D; g.row0 = row_begin; g.row_end = row_end; g.metric = metric;
    g.neg_c_log2e = 0.f; g.tau2 = -1.f;
    g.w = w; g.a = a; g.sim_out = out; g.status = reinterpret_cast<int*>(ws);
    return launch_gram<MODE_SIM>(feat, g, stream, true, nullptr);
}

}  // namespace vitcop
