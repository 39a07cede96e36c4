// Cluster merge (Eq. 6 / second half of Algorithm 3): the tokens of a cluster that were not kept as elites are
// averaged into one representative row.
//
// Two kernels on one stream:
//   merge_plan_kernel   one CTA per sample: counts the non-elite tokens of every label value in shared memory and
//                       lists the clusters that have some, in ascending label order (ordered ballot/popc compaction)
//   merge_rows_kernel   one CTA per (merged row, sample, slice of the hidden dimension): collects the members of its
//                       cluster in ascending token order, then streams their hidden rows with 128-bit loads and sums
//                       them in fp32 in that fixed order (bit-reproducible); only rows that are averaged are read.
#include <cuda_bf16.h>

#include "internal.cuh"

namespace vitcop {
namespace {

constexpr int kPlanThreads = 1024;
constexpr int kRowsThreads = 256;

// Exclusive prefix count of `flag` over the CTA in thread order; `total` receives the CTA-wide count.
template <int THREADS>
__device__ __forceinline__ uint32_t cta_prefix_count(bool flag, uint32_t* warp_sums, uint32_t& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t bal = __ballot_sync(0xffffffffu, flag);
    const uint32_t before = __popc(bal & ((1u << lane) - 1u));
    if (lane == 0) warp_sums[warp] = __popc(bal);
    __syncthreads();
    uint32_t v = lane < THREADS / 32 ? warp_sums[lane] : 0u;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, v, off);
        if (lane >= off) v += t;
    }
    total = __shfl_sync(0xffffffffu, v, THREADS / 32 - 1);
    const uint32_t base = warp == 0 ? 0u : __shfl_sync(0xffffffffu, v, warp - 1);
    __syncthreads();
    return base + before;
}

__global__ void __launch_bounds__(kPlanThreads)
merge_plan_kernel(const int32_t* __restrict__ label, const uint8_t* __restrict__ keep_mask,
                  const int32_t* __restrict__ vis_len, int vis_len_uniform, int Nv_cap, int Mcap,
                  int32_t* __restrict__ merged_label, int32_t* __restrict__ merged_count,
                  int32_t* __restrict__ n_merged) {
    extern __shared__ __align__(16) uint32_t cnt[];       // [n] non-elite tokens per label value
    __shared__ uint32_t warp_sums[32];
    grid_dependency_wait();
    const int b = blockIdx.x, tid = threadIdx.x;
    int n = vis_len ? vis_len[b] : vis_len_uniform;
    n = max(0, min(n, Nv_cap));
    label += (size_t)b * Nv_cap;
    keep_mask += (size_t)b * Nv_cap;
    merged_label += (size_t)b * Mcap;
    merged_count += (size_t)b * Mcap;
    for (int i = tid; i < n; i += kPlanThreads) cnt[i] = 0;
    __syncthreads();
    for (int i = tid; i < n; i += kPlanThreads) {
        if (keep_mask[i]) continue;
        uint32_t lab = (uint32_t)label[i];
        if (lab >= (uint32_t)n) lab = (uint32_t)n - 1;     // out-of-range labels are clamped, never indexed
        atomicAdd(&cnt[lab], 1u);
    }
    __syncthreads();
    uint32_t running = 0;
    for (int base = 0; base < n; base += kPlanThreads) {
        const int l = base + tid;
        const uint32_t c = l < n ? cnt[l] : 0u;
        uint32_t total;
        const uint32_t slot = running + cta_prefix_count<kPlanThreads>(c > 0, warp_sums, total);
        if (c > 0 && slot < (uint32_t)Mcap) {
            merged_label[slot] = l;
            merged_count[slot] = (int32_t)c;
        }
        running += total;
    }
    if (tid == 0) n_merged[b] = (int32_t)running;
    grid_dependency_launch_dependents();
}

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void add8(float (&a)[8], const uint4& v) {
    a[0] += bf16lo(v.x); a[1] += bf16hi(v.x); a[2] += bf16lo(v.y); a[3] += bf16hi(v.y);
    a[4] += bf16lo(v.z); a[5] += bf16hi(v.z); a[6] += bf16lo(v.w); a[7] += bf16hi(v.w);
}

__global__ void __launch_bounds__(kRowsThreads)
merge_rows_kernel(const uint4* __restrict__ hidden, int N, int dh8, int vis_start, const int32_t* __restrict__ label,
                  const uint8_t* __restrict__ keep_mask, const int32_t* __restrict__ vis_len, int vis_len_uniform,
                  int Nv_cap, int Mcap, const int32_t* __restrict__ merged_label,
                  const int32_t* __restrict__ merged_count, const int32_t* __restrict__ n_merged,
                  uint4* __restrict__ merged_bf16, float* __restrict__ merged_f32) {
    extern __shared__ __align__(16) uint16_t members[];   // token indices of this cluster's non-elite tokens, ascending
    __shared__ uint32_t warp_sums[32];
    grid_dependency_wait();
    const int m = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
    if (m >= min(n_merged[b], Mcap)) return;
    int n = vis_len ? vis_len[b] : vis_len_uniform;
    n = max(0, min(n, Nv_cap));
    const int lab = merged_label[(size_t)b * Mcap + m];
    const int count = merged_count[(size_t)b * Mcap + m];
    label += (size_t)b * Nv_cap;
    keep_mask += (size_t)b * Nv_cap;

    uint32_t running = 0;
    for (int base = 0; base < n; base += kRowsThreads) {
        const int i = base + tid;
        bool mine = false;
        if (i < n && !keep_mask[i]) {
            uint32_t l = (uint32_t)label[i];
            if (l >= (uint32_t)n) l = (uint32_t)n - 1;
            mine = (int)l == lab;
        }
        uint32_t total;
        const uint32_t r = running + cta_prefix_count<kRowsThreads>(mine, warp_sums, total);
        if (mine) members[r] = (uint16_t)i;
        running += total;
        if ((int)running >= count) break;                  // uniform: every thread sees the same totals
    }
    __syncthreads();

    const int piece = blockIdx.z * kRowsThreads + tid;    // 16-byte piece of the hidden row this thread owns
    if (piece >= dh8) return;
    const uint4* src = hidden + ((size_t)b * N + vis_start) * dh8 + piece;
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    int r = 0;
    for (; r + 4 <= count; r += 4) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) v[u] = ld_stream(src + (size_t)members[r + u] * dh8);
#pragma unroll
        for (int u = 0; u < 4; ++u) add8(acc, v[u]);
    }
    for (; r < count; ++r) add8(acc, ld_stream(src + (size_t)members[r] * dh8));
    const float inv = (float)count;
#pragma unroll
    for (int u = 0; u < 8; ++u) acc[u] = acc[u] / inv;
    const size_t o = ((size_t)b * Mcap + m) * dh8 + piece;
    if (merged_f32) {
        float4* d = reinterpret_cast<float4*>(merged_f32 + o * 8);
        d[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
        d[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
    }
    if (merged_bf16) {
        uint4 w;
        __nv_bfloat162 t;
        t = __floats2bfloat162_rn(acc[0], acc[1]); w.x = *reinterpret_cast<uint32_t*>(&t);
        t = __floats2bfloat162_rn(acc[2], acc[3]); w.y = *reinterpret_cast<uint32_t*>(&t);
        t = __floats2bfloat162_rn(acc[4], acc[5]); w.z = *reinterpret_cast<uint32_t*>(&t);
        t = __floats2bfloat162_rn(acc[6], acc[7]); w.w = *reinterpret_cast<uint32_t*>(&t);
        merged_bf16[o] = w;
    }
}

}  // namespace

int launch_merge(const void* hidden, int B, int N, int Dh, int vis_start, const int32_t* vis_len, int vis_len_uniform,
                 int Nv_cap, const int32_t* label, const uint8_t* keep_mask, void* merged_bf16, float* merged_f32,
                 int32_t* merged_label, int32_t* merged_count, int32_t* n_merged, int Mcap, cudaStream_t stream) {
    if (B <= 0) return VITCOP_OK;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    {
        const size_t smem = (size_t)(Nv_cap > 0 ? Nv_cap : 1) * sizeof(uint32_t);
        if (smem > 48 * 1024) {
            cudaError_t e = cudaFuncSetAttribute(merge_plan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return record_cuda(e);
        }
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(B);
        cfg.blockDim = dim3(kPlanThreads);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = stream;
        cfg.attrs = attr;
        cfg.numAttrs = pdl_allowed(true) ? 1 : 0;
        KernelTimeScope timed("merge_plan_kernel", stream);
        int rc = record_cuda(cudaLaunchKernelEx(&cfg, merge_plan_kernel, label, keep_mask, vis_len, vis_len_uniform,
                                                Nv_cap, Mcap, merged_label, merged_count, n_merged));
        if (rc != VITCOP_OK) return rc;
    }
    if (Mcap <= 0 || Dh <= 0 || (!merged_bf16 && !merged_f32)) return VITCOP_OK;
    const int dh8 = Dh / 8;
    const size_t smem = (size_t)(Nv_cap > 0 ? Nv_cap : 1) * sizeof(uint16_t);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(Mcap, B, (dh8 + kRowsThreads - 1) / kRowsThreads);
    cfg.blockDim = dim3(kRowsThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_allowed(true) ? 1 : 0;
    KernelTimeScope timed("merge_rows_kernel", stream);
    return record_cuda(cudaLaunchKernelEx(&cfg, merge_rows_kernel, static_cast<const uint4*>(hidden), N, dh8, vis_start,
                                          label, keep_mask, vis_len, vis_len_uniform, Nv_cap, Mcap,
                                          (const int32_t*)merged_label, (const int32_t*)merged_count,
                                          (const int32_t*)n_merged, static_cast<uint4*>(merged_bf16), merged_f32));
}

}  // namespace vitcop
