// The K-norm of Eq. 4 at the source of K: the key projection K^(h) = W_k^(h) t for all heads as one bf16 GEMM on the
// tensor cores (tcgen05, fp32 accumulators in tensor memory, operands staged by TMA), with rotary position embedding,
// the bf16 rounding of K and the sum of squares of every token's K vectors in the epilogue.  The separate read of K
// that a stand-alone K-norm costs (the largest byte term of a pruning step) disappears.
//
//   A = hidden [B * N, Dh] (rows = tokens), B = W_k [H * d, Dh] (rows = output features, as a linear layer stores its
//   weight): both K-major, so D = A * B^T needs no transposition.  Output tile 128 tokens x 256 features.
//
// One persistent CTA per SM, warp-specialised like the Gram sweep: warp 0 loads, one thread of warp 1 issues the
// MMAs into one of two accumulators, 8 epilogue warps drain the other: a thread owns one token row (its TMEM lane),
// the two warps of a lane quarter share the row's 256 columns.  Per 32-column chunk a thread rounds the values to
// bf16 (round to nearest even), stores them (64 contiguous bytes of K[b, h, t, :]) and adds their squares -- of the
// ROUNDED values, i.e. Eq. 4 of the K cache as written -- to the row's fp32 partial sum.  With rotary embedding the
// chunks holding the two halves of a head are taken together and turned first.  Partial sums go to one slot per
// column tile and are added by a second, tiny kernel in slot order (the same bits on every run).
// Every wait is bounded; on expiry the CTA leaves in order and the call reports VITCOP_ERR_TIMEOUT.
#include "async_copy.cuh"
#include "gram.cuh"
#include "tcgen05.cuh"

namespace vitcop {
namespace {

constexpr int BM = 128, BN = 256;
constexpr int kStages = 4;
constexpr int kABytes = BM * BK * 2, kBBytes = BN * BK * 2, kStageBytes = kABytes + kBBytes;
constexpr int kEpiWarps = 8, kEpiThreads = kEpiWarps * 32, kThreads = 64 + kEpiThreads;
constexpr int kSmemBytes = 1024 + kStages * kStageBytes + BM * 4 + 256;

struct KprojArgs {
    int B, N, Dh, H, d;
    int M, NO;                      // rows of A (B * N), output features (H * d)
    int TI, TJ;                     // row tiles, column tiles
    uint16_t* K_out;                // bf16 [B, H, N, d]
    float* part;                    // [TJ, M] sum of squares of a token's values inside one column tile
    const float* cos_tab;           // [n_pos, d / 2] or null (no rotation)
    const float* sin_tab;
    const int32_t* position;        // [B, N] or null (token index)
    int n_pos;
    int* status;
    unsigned long long wait_ns;
};

__device__ __forceinline__ uint32_t pack_bf16_rne(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// Rounds 32 values to bf16, stores them to `dst` (64 bytes, 16-byte aligned) and returns the sum of the squares of the
// rounded values, two running sums side by side.
__device__ __forceinline__ float round_store_sumsq(const float (&v)[32], uint16_t* dst, bool write) {
    uint32_t w[16];
    float s0 = 0.f, s1 = 0.f;
#pragma unroll
    for (int u = 0; u < 16; ++u) {
        w[u] = pack_bf16_rne(v[2 * u], v[2 * u + 1]);
        const float a = bf16lo(w[u]), b = bf16hi(w[u]);
        s0 = fmaf(a, a, s0);
        s1 = fmaf(b, b, s1);
    }
    if (write) {
        uint4* o = reinterpret_cast<uint4*>(dst);
#pragma unroll
        for (int q = 0; q < 4; ++q) o[q] = make_uint4(w[4 * q], w[4 * q + 1], w[4 * q + 2], w[4 * q + 3]);
    }
    return s0 + s1;
}

template <bool ROPE>
__global__ void __launch_bounds__(kThreads, 1)
kproj_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const KprojArgs k) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;
    uint8_t* gen = smem_raw + (tiles - raw);
    float* rowsum = reinterpret_cast<float*>(gen + kStages * kStageBytes);           // [BM] second slice's partial
    uint64_t* bars = reinterpret_cast<uint64_t*>(gen + kStages * kStageBytes + BM * 4);
    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * kStages;
    const uint32_t bar_tfull = bar_empty + 8 * kStages, bar_tempty = bar_tfull + 16, bar_drain = bar_tempty + 16;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStages + 5);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr uint32_t kTmemCols = 2 * BN;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
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

    const long long total = (long long)k.TI * k.TJ;
    const int KB = k.Dh / BK;
    uint32_t issued = 0, issued_parity = 0;                // thread 0, per stage: a load was issued / parity of its phase

    // Everything this kernel reads may come from the kernel before it on the stream.
    grid_dependency_wait();

    if (warp == 0) {
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            for (long long t = blockIdx.x; ok && t < total; t += gridDim.x) {
                const int ti = (int)(t / k.TJ), tj = (int)(t - (long long)ti * k.TJ);
                for (int kb = 0; kb < KB; ++kb) {
                    if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, k.wait_ns)) { ok = false; break; }
                    const uint32_t sa = tiles + stage * kStageBytes;
                    mbar_expect_tx(bar_full + 8 * stage, kStageBytes);     // rows outside the tensors arrive as zeros
                    tma_load_3d(sa, &map_a, bar_full + 8 * stage, kb * BK, ti * BM, 0);
                    tma_load_3d(sa + kABytes, &map_b, bar_full + 8 * stage, kb * BK, tj * BN, 0);
                    issued |= 1u << stage;
                    issued_parity = (issued_parity & ~(1u << stage)) | (phase << stage);
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(BM, BN);
            uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
            bool ok = true;
            for (long long t = blockIdx.x; ok && t < total; t += gridDim.x) {
                if (!mbar_wait(bar_tempty + 8 * acc, acc_phase ^ 1u, abort_flag, k.wait_ns)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * BN;
                for (int kb = 0; kb < KB; ++kb) {
                    if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag, k.wait_ns)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = tiles + stage * kStageBytes;
                    const uint64_t da = umma_desc_k128(sa), db = umma_desc_k128(sa + kABytes);
#pragma unroll
                    for (int kk = 0; kk < BK / UMMA_K; ++kk)
                        tc_mma_bf16(d_tmem, da + (uint64_t)(2 * kk), db + (uint64_t)(2 * kk), idesc,
                                    (kb > 0 || kk > 0) ? 1u : 0u);
                    tc_commit(bar_empty + 8 * stage);
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                tc_commit(bar_tfull + 8 * acc);
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
            if (!ok) {
                tc_commit(bar_drain);
                mbar_drain(bar_drain, 0);
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue
        const int quarter = warp & 3, slice = (warp - 2) >> 2;     // TMEM lane quarter; which chunks of the row
        const int rl = quarter * 32 + lane;
        const int half32 = k.d / 64;                               // chunks in half a head (rotation only)
        uint32_t acc = 0, acc_phase = 0;
        bool ok = true;
        for (long long t = blockIdx.x; t < total; t += gridDim.x) {
            const int ti = (int)(t / k.TJ), tj = (int)(t - (long long)ti * k.TJ);
            const int m = ti * BM + rl;                            // token row of this thread
            const bool row_valid = m < k.M;
            const int b = row_valid ? m / k.N : 0, tok = row_valid ? m - b * k.N : 0;
            if (ok) ok = mbar_wait(bar_tfull + 8 * acc, acc_phase, abort_flag, k.wait_ns);
            ok = __all_sync(0xffffffffu, ok);
            float ssq = 0.f;
            if (ok) {
                tc_fence_after();
                const uint32_t taddr = tmem_base + acc * BN + ((uint32_t)(quarter * 32) << 16);
                auto dst_of = [&](int chunk) -> uint16_t* {        // K[b, head, tok, e0 ..] of a 32-column chunk
                    const int col = tj * BN + chunk * 32;
                    const int head = col / k.d, e0 = col - head * k.d;
                    return k.K_out + (((size_t)b * k.H + head) * k.N + tok) * k.d + e0;
                };
                if (!ROPE) {
#pragma unroll 1
                    for (int c = 0; c < 4; ++c) {
                        const int chunk = slice * 4 + c;
                        float v[32];
                        tmem_ld32(taddr + chunk * 32, v);
                        const bool write = row_valid && tj * BN + chunk * 32 < k.NO;
                        ssq += round_store_sumsq(v, dst_of(chunk), write);
                    }
                } else {
                    // pairs of chunks that hold columns e and e + d / 2 of one head: two per slice
                    const int p = row_valid ? (k.position ? k.position[(size_t)b * k.N + tok] : tok) : 0;
                    const int pos = min(max(p, 0), k.n_pos - 1);
#pragma unroll 1
                    for (int c = 0; c < 2; ++c) {
                        const int q = slice * 2 + c;                               // pair number inside the tile
                        const int lo = (q / half32) * 2 * half32 + q % half32, hi = lo + half32;
                        float x[32], y[32];
                        tmem_ld32(taddr + lo * 32, x);
                        tmem_ld32(taddr + hi * 32, y);
                        const int e0 = (tj * BN + lo * 32) % k.d;                  // first of the 32 rotation angles
                        const float4* ct = reinterpret_cast<const float4*>(k.cos_tab + (size_t)pos * (k.d / 2) + e0);
                        const float4* st = reinterpret_cast<const float4*>(k.sin_tab + (size_t)pos * (k.d / 2) + e0);
#pragma unroll
                        for (int u4 = 0; u4 < 8; ++u4) {
                            const float4 cc = __ldg(ct + u4), ss = __ldg(st + u4);
                            const float cv[4] = {cc.x, cc.y, cc.z, cc.w}, sv[4] = {ss.x, ss.y, ss.z, ss.w};
#pragma unroll
                            for (int r = 0; r < 4; ++r) {
                                const float a = x[4 * u4 + r], bb = y[4 * u4 + r];
                                x[4 * u4 + r] = fmaf(a, cv[r], -(bb * sv[r]));
                                y[4 * u4 + r] = fmaf(bb, cv[r], a * sv[r]);
                            }
                        }
                        const bool write = row_valid && tj * BN + hi * 32 < k.NO;
                        ssq += round_store_sumsq(x, dst_of(lo), write);
                        ssq += round_store_sumsq(y, dst_of(hi), write);
                    }
                }
                tc_fence_before();
                mbar_arrive(bar_tempty + 8 * acc);
            }
            // the row's two slices meet in shared memory; slice 0 writes the tile's partial sum
            if (slice == 1) rowsum[rl] = ssq;
            epi_bar_sync<kEpiThreads>();
            if (ok && slice == 0 && row_valid) k.part[(size_t)tj * k.M + m] = ssq + rowsum[rl];
            if (epi_bar_or<kEpiThreads>(!ok)) break;
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
        for (int s = 0; s < kStages; ++s)
            if (issued >> s & 1u) mbar_drain(bar_full + 8 * s, issued_parity >> s & 1u);
        if (k.status) atomicMax(k.status, VITCOP_ERR_TIMEOUT);
    }
    grid_dependency_launch_dependents();
}

// score[b, i] = sqrt( sum over the column tiles, in order, of the partial sums of token vis_start + i ).
__global__ void kproj_score_kernel(const float* __restrict__ part, int M, int TJ, int N, int vis_start, int Nv,
                                   float* __restrict__ score) {
    grid_dependency_wait();
    const int i = blockIdx.x * blockDim.x + threadIdx.x, b = blockIdx.y;
    if (i >= Nv) return;
    const size_t m = (size_t)b * N + vis_start + i;
    float s = 0.f;
    for (int tj = 0; tj < TJ; ++tj) s += part[(size_t)tj * M + m];
    score[(size_t)b * Nv + i] = sqrtf(s);
}

}  // namespace

size_t kproj_workspace_bytes(int B, int N, int H, int d) {
    const size_t TJ = ((size_t)H * d + BN - 1) / BN;
    return kStatusBytes + align_up(TJ * (size_t)B * N * sizeof(float), 256);
}

int launch_kproj_knorm(const void* hidden, const void* W, int B, int N, int Dh, int H, int d, const float* cos_tab,
                       const float* sin_tab, const int32_t* position, int n_pos, void* K_out, int vis_start, int Nv,
                       float* score, void* workspace, cudaStream_t stream) {
    KprojArgs k = {};
    k.B = B; k.N = N; k.Dh = Dh; k.H = H; k.d = d;
    k.M = B * N; k.NO = H * d;
    k.TI = (k.M + BM - 1) / BM; k.TJ = (k.NO + BN - 1) / BN;
    k.K_out = static_cast<uint16_t*>(K_out);
    k.part = reinterpret_cast<float*>(static_cast<char*>(workspace) + kStatusBytes);
    k.cos_tab = cos_tab; k.sin_tab = sin_tab; k.position = position; k.n_pos = n_pos;
    k.status = static_cast<int*>(workspace);
    k.wait_ns = gram_wait_limit_ns();
    const long long total = (long long)k.TI * k.TJ;
    if (total <= 0) return VITCOP_OK;
    CUtensorMap ma, mb;
    if (!make_rowmajor_bf16_map(&ma, hidden, 1, k.M, Dh, BM) || !make_rowmajor_bf16_map(&mb, W, 1, k.NO, Dh, BN))
        return VITCOP_ERR_CUDA;
    const bool rope = cos_tab != nullptr;
    auto kern = rope ? kproj_kernel<true> : kproj_kernel<false>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return record_cuda(e);
    cudaLaunchConfig_t cfg = {};
    const int sms = gram_num_sms();
    cfg.gridDim = dim3((unsigned)(total < sms ? total : sms));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = stream;
    int rc;
    {
        KernelTimeScope timed("kproj_kernel", stream);
        rc = record_cuda(cudaLaunchKernelEx(&cfg, kern, ma, mb, k));
    }
    if (rc != VITCOP_OK || Nv <= 0 || !score) return rc;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t c2 = {};
    c2.gridDim = dim3((Nv + 255) / 256, B);
    c2.blockDim = dim3(256);
    c2.stream = stream;
    c2.attrs = attr;
    c2.numAttrs = pdl_allowed(true) ? 1 : 0;
    KernelTimeScope timed("kproj_score_kernel", stream);
    return record_cuda(cudaLaunchKernelEx(&c2, kproj_score_kernel, (const float*)k.part, k.M, k.TJ, N, vis_start, Nv,
                                          score));
}

}  // namespace vitcop
