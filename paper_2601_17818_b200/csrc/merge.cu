// Cluster merge (Eq. 6 / second half of Algorithm 3): the tokens of a cluster that were not kept as elites are
// averaged into one representative row.
//
// Two kernels on one stream:
//   merge_plan_kernel   one CTA per sample: sorts the (label, token index) pairs of the non-elite tokens in shared
//                       memory, which lays every cluster's members out contiguously in ascending token order; the
//                       clusters that have members are numbered in ascending label order (ordered ballot/popc
//                       compaction of the run heads) and the member list goes to the workspace
//   merge_rows_kernel   one CTA per (merged row, sample, 512-byte slice of the hidden row): its eight warps stream
//                       the members' row slices with 128-bit loads (member r goes to warp r mod 8) and the eight
//                       fp32 partial sums are added in warp order, a fixed order (bit-reproducible).  Only rows
//                       that are averaged are read.
#include <cuda_bf16.h>

#include "block_sort.cuh"
#include "internal.cuh"

namespace vitcop {
namespace {

constexpr int kPlanThreads = 1024;
constexpr int kRowsThreads = 256;

// Loads the keys (label << 32 | index) of the non-elite tokens, ~0 for everything else, and sorts them.
template <int E>
__device__ void sort_members(const int32_t* __restrict__ label, const uint8_t* __restrict__ keep_mask, int n, int T,
                             unsigned long long* comp) {
    unsigned long long r[E];
    const int t = threadIdx.x;
#pragma unroll
    for (int e = 0; e < E; ++e) {
        const int i = t * E + e;
        unsigned long long c = ~0ull;
        if (t < T && i < n && !keep_mask[i]) {
            uint32_t lab = (uint32_t)label[i];
            if (lab >= (uint32_t)n) lab = (uint32_t)n - 1;          // out-of-range labels are clamped, never indexed
            c = ((unsigned long long)lab << 32) | (unsigned long long)i;
        }
        r[e] = c;
    }
    block_bitonic_sort<E>(r, comp, T);
}

__global__ void __launch_bounds__(kPlanThreads)
merge_plan_kernel(const int32_t* __restrict__ label, const uint8_t* __restrict__ keep_mask,
                  const int32_t* __restrict__ vis_len, int vis_len_uniform, int Nv_cap, int Mcap,
                  int32_t* __restrict__ merged_label, int32_t* __restrict__ merged_count,
                  int32_t* __restrict__ n_merged, uint16_t* __restrict__ members, int32_t* __restrict__ starts) {
    extern __shared__ __align__(16) unsigned long long comp[];   // [P] sorted keys
    __shared__ uint32_t warp_sums[32];
    grid_dependency_wait();
    const int b = blockIdx.x, tid = threadIdx.x;
    int n = vis_len ? vis_len[b] : vis_len_uniform;
    n = max(0, min(n, Nv_cap));
    label += (size_t)b * Nv_cap;
    keep_mask += (size_t)b * Nv_cap;
    merged_label += (size_t)b * Mcap;
    merged_count += (size_t)b * Mcap;
    members += (size_t)b * Nv_cap;
    starts += (size_t)b * Mcap;

    int P = 256;                                          // at least one warp of 8 keys per thread
    while (P < n) P <<= 1;
    if (P <= 8 * kPlanThreads) sort_members<8>(label, keep_mask, n, P / 8, comp);
    else sort_members<16>(label, keep_mask, n, P / 16, comp);

    // run heads -> merged rows (ascending label); run tails close them; the sorted indices are the member list
    uint32_t heads = 0, tails = 0;
    for (int base = 0; base < P; base += kPlanThreads) {
        const int p = base + tid;
        const unsigned long long c = p < n ? comp[p] : ~0ull;     // non-elite tokens sort to the front, at most n of them
        const bool valid = c != ~0ull;
        const uint32_t lab = (uint32_t)(c >> 32);
        const bool head = valid && (p == 0 || (uint32_t)(comp[p - 1] >> 32) != lab);
        const bool tail = valid && (p + 1 >= n || comp[p + 1] == ~0ull || (uint32_t)(comp[p + 1] >> 32) != lab);
        if (valid) members[p] = (uint16_t)(c & 0xFFFFull);
        uint32_t th, tt;
        const uint32_t hs = heads + block_prefix_count(head, warp_sums, th);
        const uint32_t ts = tails + block_prefix_count(tail, warp_sums, tt);
        if (head && hs < (uint32_t)Mcap) {
            merged_label[hs] = (int32_t)lab;
            starts[hs] = p;
        }
        if (tail && ts < (uint32_t)Mcap) merged_count[ts] = p;          // position of the run's last member for now
        heads += th;
        tails += tt;
        if (base + kPlanThreads >= n) break;                            // uniform
    }
    __syncthreads();
    for (int m = tid; m < min((int)heads, Mcap); m += kPlanThreads) merged_count[m] = merged_count[m] - starts[m] + 1;
    if (tid == 0) n_merged[b] = (int32_t)heads;
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
merge_rows_kernel(const uint4* __restrict__ hidden, int N, int dh8, int vis_start, int Nv_cap, int Mcap,
                  const int32_t* __restrict__ merged_count, const int32_t* __restrict__ n_merged,
                  const uint16_t* __restrict__ members, const int32_t* __restrict__ starts,
                  void* __restrict__ merged_bf16, float* __restrict__ merged_f32) {
    constexpr int G = kRowsThreads / 32;                  // warps sharing the members
    __shared__ float partial[G][32][9];                   // padded against bank conflicts
    grid_dependency_wait();
    const int m = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
    // the three descriptors of the row are independent loads: issue them together
    const int nm = n_merged[b];
    const int count = merged_count[(size_t)b * Mcap + m];
    const int start = starts[(size_t)b * Mcap + m];
    if (m >= min(nm, Mcap)) return;
    const uint16_t* mem = members + (size_t)b * Nv_cap + start;

    const int g = tid >> 5, lane = tid & 31;
    const int piece = blockIdx.z * 32 + lane;             // 16-byte piece of the hidden row this lane owns
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    if (piece < dh8) {
        const uint4* src = hidden + ((size_t)b * N + vis_start) * dh8 + piece;
        int r = g;
        for (; r + 3 * G < count; r += 4 * G) {
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) v[u] = ld_stream(src + (size_t)mem[r + u * G] * dh8);
#pragma unroll
            for (int u = 0; u < 4; ++u) add8(acc, v[u]);
        }
        for (; r < count; r += G) add8(acc, ld_stream(src + (size_t)mem[r] * dh8));
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) partial[g][lane][u] = acc[u];
    __syncthreads();
    const int pl = tid & 31, k = tid >> 5;                // this thread finishes element k of piece pl
    const int pcol = blockIdx.z * 32 + pl;
    if (pcol >= dh8) return;
    float sum = 0.f;
#pragma unroll
    for (int q = 0; q < G; ++q) sum += partial[q][pl][k];   // warp order: fixed
    sum = sum / (float)count;
    const size_t o = (((size_t)b * Mcap + m) * dh8 + pcol) * 8 + k;
    if (merged_f32) merged_f32[o] = sum;
    if (merged_bf16) static_cast<__nv_bfloat16*>(merged_bf16)[o] = __float2bfloat16_rn(sum);
}

// Workspace: status | members uint16 [B, Nv_cap] | starts int32 [B, Mcap]
struct MergeWs {
    size_t off_members, off_starts, total;
    MergeWs(int B, int Nv_cap, int Mcap) {
        size_t o = kStatusBytes;
        off_members = o; o += align_up((size_t)B * Nv_cap * sizeof(uint16_t), 256);
        off_starts = o;  o += align_up((size_t)B * Mcap * sizeof(int32_t), 256);
        total = o;
    }
};

}  // namespace

size_t merge_workspace_bytes(int B, int Nv_cap, int Mcap) { return MergeWs(B, Nv_cap, Mcap).total; }

int launch_merge(const void* hidden, int B, int N, int Dh, int vis_start, const int32_t* vis_len, int vis_len_uniform,
                 int Nv_cap, const int32_t* label, const uint8_t* keep_mask, void* merged_bf16, float* merged_f32,
                 int32_t* merged_label, int32_t* merged_count, int32_t* n_merged, int Mcap, void* workspace,
                 cudaStream_t stream) {
    if (B <= 0) return VITCOP_OK;
    const MergeWs lay(B, Nv_cap, Mcap);
    char* ws = static_cast<char*>(workspace);
    uint16_t* members = reinterpret_cast<uint16_t*>(ws + lay.off_members);
    int32_t* starts = reinterpret_cast<int32_t*>(ws + lay.off_starts);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    {
        int P = 256;
        while (P < Nv_cap) P <<= 1;
        const size_t smem = (size_t)P * sizeof(unsigned long long);
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
                                                Nv_cap, Mcap, merged_label, merged_count, n_merged, members, starts));
        if (rc != VITCOP_OK) return rc;
    }
    if (Mcap <= 0 || Dh <= 0 || (!merged_bf16 && !merged_f32)) return VITCOP_OK;
    const int dh8 = Dh / 8;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(Mcap, B, (dh8 + 31) / 32);
    cfg.blockDim = dim3(kRowsThreads);
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_allowed(true) ? 1 : 0;
    KernelTimeScope timed("merge_rows_kernel", stream);
    return record_cuda(cudaLaunchKernelEx(&cfg, merge_rows_kernel, static_cast<const uint4*>(hidden), N, dh8, vis_start,
                                          Nv_cap, Mcap, (const int32_t*)merged_count, (const int32_t*)n_merged,
                                          (const uint16_t*)members, (const int32_t*)starts, merged_bf16, merged_f32));
}

}  // namespace vitcop
