// K-norm saliency (Eq. 4): score_i = sqrt( sum_h sum_e K[b,h,i,e]^2 ) over the visual span.
//
// HBM-bound streaming reduction.  A group of LPR consecutive lanes owns one token: every lane
// issues 128-bit loads (8 bf16) from the token's row in each head, squares in fp32 (a bf16
// product is exact in fp32), accumulates over heads in registers and the group finishes with
// xor-shuffles.  Consecutive tokens of one head are contiguous in memory, so a CTA's loads of one
// head form one contiguous run of TOKENS_PER_CTA * d * 2 bytes.
#include "knorm.cuh"

namespace vitcop {
namespace {

constexpr int kKnormThreads = 128;

// Strides are in units of 16 bytes (8 elements).
template <int LPR, int UNROLL>
__global__ void __launch_bounds__(kKnormThreads)
knorm_kernel(const uint4* __restrict__ K, int H, int d8, int64_t sb, int64_t sh, int64_t sn, int vis_start,
             const int32_t* __restrict__ vis_len, int vis_len_uniform, float* __restrict__ score, int Nv_cap,
             int late_wait) {
    // late_wait: K is known to be final already (the caller ordered its producer before the preceding grid), so
    // this grid may run beside the preceding one; it still waits for it before it ends, which keeps "this grid
    // has completed" meaning "everything before it has completed" for the kernels that follow.
    if (!late_wait) grid_dependency_wait();
    const int b = blockIdx.y;
    // a device-side length never reaches past the capacity of the score row (nor, the host has checked, of K)
    const int nv = max(0, min(vis_len ? vis_len[b] : vis_len_uniform, Nv_cap));
    constexpr int kTok = kKnormThreads / LPR;
    const int sub = threadIdx.x % LPR;
    const int i = blockIdx.x * kTok + threadIdx.x / LPR;
    float acc = 0.f;
    if (i < nv)
        acc = knorm_token_partial<LPR, UNROLL>(K + b * sb + (int64_t)(vis_start + i) * sn, H, d8, sh, sub);
#pragma unroll
    for (int off = LPR / 2; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if (i < nv && sub == 0) score[(int64_t)b * Nv_cap + i] = sqrtf(acc);
    // Only now may the next kernel's CTAs be scheduled: released earlier they would sit on the SMs waiting for
    // this grid while its own remaining CTAs queue behind them.
    grid_dependency_launch_dependents();
    // One waiting CTA is enough to keep the grid from completing early; the others leave and free their SM slots
    // for the CTAs of this grid that have not started yet.
    if (late_wait && blockIdx.x == 0 && blockIdx.y == 0) grid_dependency_wait();
}

}  // namespace

int launch_knorm(const void* K, int B, int H, int d, int64_t stride_b, int64_t stride_h, int64_t stride_n,
                 int vis_start, const int32_t* vis_len, int vis_len_uniform, float* score, int Nv_cap,
                 cudaStream_t stream, bool late_wait, bool* launched) {
    if (launched) *launched = false;
    if (B <= 0 || Nv_cap <= 0 || H <= 0) return VITCOP_OK;
    const int d8 = d / 8;
    const int span = vis_len ? Nv_cap : vis_len_uniform;
    if (span <= 0) return VITCOP_OK;
    if (launched) *launched = true;
    const uint4* Kp = static_cast<const uint4*>(K);
    const int64_t sb = stride_b / 8, sh = stride_h / 8, sn = stride_n / 8;
    int rc = VITCOP_OK;
    auto go = [&](auto kern, int lpr) {
        const int tok = kKnormThreads / lpr;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((span + tok - 1) / tok, B);
        cfg.blockDim = dim3(kKnormThreads);
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = pdl_allowed(true) ? 1 : 0;
        KernelTimeScope timed("knorm_kernel", stream);
        rc = record_cuda(cudaLaunchKernelEx(&cfg, kern, Kp, H, d8, sb, sh, sn, vis_start, vis_len, vis_len_uniform,
                                            score, Nv_cap, late_wait ? 1 : 0));
    };
    if (d8 >= 16) go(knorm_kernel<16, 8>, 16);
    else if (d8 >= 8) go(knorm_kernel<8, 8>, 8);
    else if (d8 >= 4) go(knorm_kernel<4, 8>, 4);
    else go(knorm_kernel<1, 8>, 1);
    return rc;
}

}  // namespace vitcop
