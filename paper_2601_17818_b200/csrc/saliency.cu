// Stage I saliency (Eq. 1): S_i = sum_h A^(h)_{0,i}, the attention the [CLS] query pays to visual token i,
// summed over the heads of the vision-encoder layer.
//
//   cls_logits_kernel     one CTA per (chunk of 256 keys, head, image): logits scale * q . k_j, a key row spread over
//                         8, 16 or 32 lanes (one 128-bit load per lane and piece, rows of a warp side by side in
//                         memory), several rows in flight per lane; logits to the workspace [B, H, M] together with
//                         the chunk's maximum and its sum of exp(logit - maximum)
//   cls_saliency_kernel   per (image, block of keys): the softmax denominators of all heads from the chunk partials
//                         (fixed order), then S[b, j-1] = sum over heads, in head order, of exp(logit - max) / den
// HBM traffic is the key tensor, read once (the logits are 4 bytes per key row, written and read once).
#include "internal.cuh"

namespace vitcop {
namespace {

constexpr int kSalThreads = 256;
constexpr int kSalChunk = 256;                             // keys per CTA of the first kernel
constexpr int kSalWarps = kSalThreads / 32;
constexpr int kSalHeadLanes = 4;                           // threads that share a key's heads in the second kernel
constexpr int kSalKeys = kSalThreads / kSalHeadLanes;      // keys per CTA of the second kernel

// Block-wide maximum or sum in a fixed order; every thread gets the result.
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
    for (int w = 1; w < kSalWarps; ++w) r = is_max ? fmaxf(r, scratch[w]) : r + scratch[w];
    return r;
}

__device__ __forceinline__ void dot8(const uint4& k, const float* q, float& a0, float& a1) {
    a0 = fmaf(bf16lo(k.x), q[0], a0); a1 = fmaf(bf16hi(k.x), q[1], a1);
    a0 = fmaf(bf16lo(k.y), q[2], a0); a1 = fmaf(bf16hi(k.y), q[3], a1);
    a0 = fmaf(bf16lo(k.z), q[4], a0); a1 = fmaf(bf16hi(k.z), q[5], a1);
    a0 = fmaf(bf16lo(k.w), q[6], a0); a1 = fmaf(bf16hi(k.w), q[7], a1);
}

// LANES lanes share a key row: lane `sub` takes the 16-byte pieces sub, sub + LANES, ..
template <int LANES>
__global__ void __launch_bounds__(kSalThreads)
cls_logits_kernel(const uint4* __restrict__ q, const uint4* __restrict__ K, int H, int M, int d8, float scale_log2e,
                  float* __restrict__ logit, float2* __restrict__ part) {
    constexpr int kRowsPerPass = kSalThreads / LANES;
    constexpr int kPasses = kSalChunk / kRowsPerPass;      // == LANES
    constexpr int kInFlight = 4;                           // rows a lane requests before it reduces any
    extern __shared__ __align__(16) float qs[];            // the query row as fp32 [8 * d8]
    __shared__ float lg[kSalChunk];
    __shared__ float scratch[kSalWarps];
    grid_dependency_wait();
    const int chunk = blockIdx.x, h = blockIdx.y, b = blockIdx.z, tid = threadIdx.x;
    const int chunks = gridDim.x;
    const int sub = tid % LANES, slot = tid / LANES;
    const uint4* qrow = q + ((size_t)b * H + h) * d8;
    for (int c = tid; c < d8; c += kSalThreads) {
        const uint4 v = qrow[c];
        float* o = qs + c * 8;
        o[0] = bf16lo(v.x); o[1] = bf16hi(v.x); o[2] = bf16lo(v.y); o[3] = bf16hi(v.y);
        o[4] = bf16lo(v.z); o[5] = bf16hi(v.z); o[6] = bf16lo(v.w); o[7] = bf16hi(v.w);
    }
    __syncthreads();
    const bool one_piece = d8 <= LANES;                    // the usual case: the lane's part of q stays in registers
    float qr[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) qr[u] = (one_piece && sub < d8) ? qs[sub * 8 + u] : 0.f;

    const int j0 = chunk * kSalChunk;
    const uint4* Kh = K + ((size_t)b * H + h) * M * d8;
#pragma unroll 1
    for (int p0 = 0; p0 < kPasses; p0 += kInFlight) {
        float acc[kInFlight];
        if (one_piece) {
            uint4 kv[kInFlight];
#pragma unroll
            for (int u = 0; u < kInFlight; ++u) {
                const int j = j0 + (p0 + u) * kRowsPerPass + slot;
                kv[u] = (j < M && sub < d8) ? Kh[(size_t)j * d8 + sub] : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int u = 0; u < kInFlight; ++u) {
                float a0 = 0.f, a1 = 0.f;
                dot8(kv[u], qr, a0, a1);
                acc[u] = a0 + a1;
            }
        } else {
#pragma unroll
            for (int u = 0; u < kInFlight; ++u) {
                const int j = j0 + (p0 + u) * kRowsPerPass + slot;
                float a0 = 0.f, a1 = 0.f;
                if (j < M)
                    for (int c = sub; c < d8; c += LANES) dot8(Kh[(size_t)j * d8 + c], qs + c * 8, a0, a1);
                acc[u] = a0 + a1;
            }
        }
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) {
#pragma unroll
            for (int off = LANES / 2; off > 0; off >>= 1) acc[u] += __shfl_xor_sync(0xffffffffu, acc[u], off);
            // logit in units of log2 e, so that exp is one ex2
            if (sub == 0) lg[(p0 + u) * kRowsPerPass + slot] = acc[u] * scale_log2e;
        }
    }
    __syncthreads();
    const int j = j0 + tid;                                // kSalChunk == kSalThreads: one key per thread
    const float l = j < M ? lg[tid] : -__builtin_huge_valf();
    const float mx = block_reduce(l, true, scratch);
    const float s = block_reduce(j < M ? exp2f(l - mx) : 0.f, false, scratch);
    if (j < M) logit[((size_t)b * H + h) * M + j] = l;
    if (tid == 0) part[((size_t)b * H + h) * chunks + chunk] = make_float2(mx, s);
    grid_dependency_launch_dependents();
}
static_assert(kSalChunk == kSalThreads, "one key per thread in the chunk reductions");

__global__ void __launch_bounds__(kSalThreads)
cls_saliency_kernel(const float* __restrict__ logit, const float2* __restrict__ part, int H, int M, int chunks,
                    float* __restrict__ saliency, float* __restrict__ cls_self) {
    extern __shared__ float hm[];                          // per head: maximum [H], denominator [H]
    float* hden = hm + H;
    grid_dependency_wait();
    const int b = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int h = warp; h < H; h += kSalWarps) {
        const float2* p = part + ((size_t)b * H + h) * chunks;
        float mx = -__builtin_huge_valf();
        for (int c = lane; c < chunks; c += 32) mx = fmaxf(mx, p[c].x);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
        float den = 0.f;
        for (int c = lane; c < chunks; c += 32) den += p[c].y * exp2f(p[c].x - mx);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) den += __shfl_xor_sync(0xffffffffu, den, off);
        if (lane == 0) { hm[h] = mx; hden[h] = den; }
    }
    __syncthreads();
    // kSalKeys keys per CTA; the heads of a key are shared out over kSalHeadLanes threads (head h to thread h mod 4,
    // in ascending order), whose partial sums are added in thread order
    const int jj = tid % kSalKeys, hg = tid / kSalKeys;
    const int j = blockIdx.x * kSalKeys + jj;
    float s = 0.f;
    if (j < M) {
        const float* l = logit + (size_t)b * H * M + j;
        for (int h = hg; h < H; h += kSalHeadLanes) s += exp2f(l[(size_t)h * M] - hm[h]) / hden[h];
    }
    __shared__ float partial[kSalHeadLanes][kSalKeys];
    partial[hg][jj] = s;
    __syncthreads();
    if (hg != 0 || j >= M) return;
#pragma unroll
    for (int g = 1; g < kSalHeadLanes; ++g) s += partial[g][jj];
    if (j == 0) {
        if (cls_self) cls_self[b] = s;
    } else {
        saliency[(size_t)b * (M - 1) + (j - 1)] = s;
    }
}

inline int sal_chunks(int M) { return (M + kSalChunk - 1) / kSalChunk; }

}  // namespace

size_t saliency_workspace_bytes(int B, int H, int M) {
    return kStatusBytes + align_up((size_t)B * H * M * 4, 256) + align_up((size_t)B * H * sal_chunks(M) * 8, 256);
}

int launch_cls_saliency(const void* q, const void* K, int B, int H, int M, int d, float scale, float* saliency,
                        float* cls_self, void* workspace, cudaStream_t stream) {
    if (B <= 0 || H <= 0 || M <= 0) return VITCOP_OK;
    if (B > 65535 || H > 4096 || d > 4096) return VITCOP_ERR_UNSUPPORTED;   // grid limits; q row and head tables in 48 KB
    const int d8 = d / 8, chunks = sal_chunks(M);
    float* logit = reinterpret_cast<float*>(static_cast<char*>(workspace) + kStatusBytes);
    float2* part = reinterpret_cast<float2*>(reinterpret_cast<char*>(logit) + align_up((size_t)B * H * M * 4, 256));
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    const size_t smem = (size_t)d * sizeof(float);
    {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(chunks, H, B);
        cfg.blockDim = dim3(kSalThreads);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = stream;
        cfg.attrs = attr;
        cfg.numAttrs = pdl_allowed(true) ? 1 : 0;
        KernelTimeScope timed("cls_logits_kernel", stream);
        auto kern = d8 <= 8 ? cls_logits_kernel<8> : d8 <= 16 ? cls_logits_kernel<16> : cls_logits_kernel<32>;
        int rc = record_cuda(cudaLaunchKernelEx(&cfg, kern, static_cast<const uint4*>(q), static_cast<const uint4*>(K),
                                                H, M, d8, scale * 1.4426950408889634f, logit, part));
        if (rc != VITCOP_OK) return rc;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((M + kSalKeys - 1) / kSalKeys, B);
    cfg.blockDim = dim3(kSalThreads);
    cfg.dynamicSmemBytes = 2 * (size_t)H * sizeof(float);
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_allowed(true) ? 1 : 0;
    KernelTimeScope timed("cls_saliency_kernel", stream);
    return record_cuda(cudaLaunchKernelEx(&cfg, cls_saliency_kernel, (const float*)logit, (const float2*)part, H, M,
                                          chunks, saliency, cls_self));
}

}  // namespace vitcop
