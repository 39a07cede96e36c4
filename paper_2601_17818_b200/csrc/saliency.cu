// Stage I saliency (Eq. 1): S_i = sum_h A^(h)_{0,i}, the attention the [CLS] query pays to visual token i,
// summed over the heads of the vision-encoder layer.
//
//   cls_attention_kernel   one CTA per (head, image): logits scale * q . k_j for all M keys (one key per
//                          thread and pass, 128-bit loads of the key row), block-wide max and sum, softmax row
//                          written to the workspace [B, H, M]
//   cls_reduce_kernel      S[b, j-1] = sum over heads in head order (fixed order: reproducible bits)
// HBM traffic is the key tensor, read once.
#include "internal.cuh"

namespace vitcop {
namespace {

constexpr int kAttnThreads = 256;

__device__ __forceinline__ float block_reduce(float v, bool is_max, float* scratch) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const float o = __shfl_xor_sync(0xffffffffu, v, off);
        v = is_max ? fmaxf(v, o) : v + o;
    }
    __syncthreads();
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    float r = scratch[0];
    for (int w = 1; w < kAttnThreads / 32; ++w) r = is_max ? fmaxf(r, scratch[w]) : r + scratch[w];   // fixed order
    return r;
}

__global__ void __launch_bounds__(kAttnThreads)
cls_attention_kernel(const uint4* __restrict__ q, const uint4* __restrict__ K, int H, int M, int d8, float scale_log2e,
                     float* __restrict__ prob) {
    extern __shared__ __align__(16) float sm[];           // q row [d] then logits [M]
    __shared__ float scratch[kAttnThreads / 32];
    grid_dependency_wait();
    const int h = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
    float* qs = sm;
    float* logit = sm + d8 * 8;
    const uint4* qrow = q + ((size_t)b * H + h) * d8;
    for (int c = tid; c < d8; c += kAttnThreads) {
        const uint4 v = qrow[c];
        float* o = qs + c * 8;
        o[0] = bf16lo(v.x); o[1] = bf16hi(v.x); o[2] = bf16lo(v.y); o[3] = bf16hi(v.y);
        o[4] = bf16lo(v.z); o[5] = bf16hi(v.z); o[6] = bf16lo(v.w); o[7] = bf16hi(v.w);
    }
    __syncthreads();
    const uint4* Kh = K + ((size_t)b * H + h) * M * d8;
    float mx = -__builtin_huge_valf();
    for (int j = tid; j < M; j += kAttnThreads) {
        const uint4* row = Kh + (size_t)j * d8;
        float a0 = 0.f, a1 = 0.f;
        for (int c = 0; c < d8; ++c) {
            const uint4 v = row[c];
            const float* qq = qs + c * 8;
            a0 = fmaf(bf16lo(v.x), qq[0], a0); a1 = fmaf(bf16hi(v.x), qq[1], a1);
            a0 = fmaf(bf16lo(v.y), qq[2], a0); a1 = fmaf(bf16hi(v.y), qq[3], a1);
            a0 = fmaf(bf16lo(v.z), qq[4], a0); a1 = fmaf(bf16hi(v.z), qq[5], a1);
            a0 = fmaf(bf16lo(v.w), qq[6], a0); a1 = fmaf(bf16hi(v.w), qq[7], a1);
        }
        const float l = (a0 + a1) * scale_log2e;          // logit in units of log2 e, so that exp is one ex2
        logit[j] = l;
        mx = fmaxf(mx, l);
    }
    mx = block_reduce(mx, true, scratch);
    float den = 0.f;
    for (int j = tid; j < M; j += kAttnThreads) {
        const float e = exp2f(logit[j] - mx);
        logit[j] = e;
        den += e;
    }
    den = block_reduce(den, false, scratch);
    float* out = prob + ((size_t)b * H + h) * M;
    for (int j = tid; j < M; j += kAttnThreads) out[j] = logit[j] / den;
    grid_dependency_launch_dependents();
}

__global__ void cls_reduce_kernel(const float* __restrict__ prob, int H, int M, float* __restrict__ saliency,
                                  float* __restrict__ cls_self) {
    grid_dependency_wait();
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    const int b = blockIdx.y;
    if (j >= M) return;
    const float* p = prob + (size_t)b * H * M + j;
    float s = 0.f;
    for (int h = 0; h < H; ++h) s += p[(size_t)h * M];
    if (j == 0) {
        if (cls_self) cls_self[b] = s;
    } else {
        saliency[(size_t)b * (M - 1) + (j - 1)] = s;
    }
}

}  // namespace

size_t saliency_workspace_bytes(int B, int H, int M) { return kStatusBytes + align_up((size_t)B * H * M * 4, 256); }

int launch_cls_saliency(const void* q, const void* K, int B, int H, int M, int d, float scale, float* saliency,
                        float* cls_self, void* workspace, cudaStream_t stream) {
    if (B <= 0 || H <= 0 || M <= 0) return VITCOP_OK;
    float* prob = reinterpret_cast<float*>(static_cast<char*>(workspace) + kStatusBytes);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    const size_t smem = ((size_t)d + M) * sizeof(float);
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(cls_attention_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return record_cuda(e);
    }
    {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(H, B);
        cfg.blockDim = dim3(kAttnThreads);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = stream;
        cfg.attrs = attr;
        cfg.numAttrs = pdl_allowed(true) ? 1 : 0;
        KernelTimeScope timed("cls_attention_kernel", stream);
        int rc = record_cuda(cudaLaunchKernelEx(&cfg, cls_attention_kernel, static_cast<const uint4*>(q),
                                                static_cast<const uint4*>(K), H, M, d / 8,
                                                scale * 1.4426950408889634f, prob));
        if (rc != VITCOP_OK) return rc;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((M + 255) / 256, B);
    cfg.blockDim = dim3(256);
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_allowed(true) ? 1 : 0;
    KernelTimeScope timed("cls_reduce_kernel", stream);
    return record_cuda(cudaLaunchKernelEx(&cfg, cls_reduce_kernel, (const float*)prob, H, M, saliency, cls_self));
}

}  // namespace vitcop
