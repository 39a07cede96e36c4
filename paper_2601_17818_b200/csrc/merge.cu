// Cluster merge (Eq. 6 / second half of Algorithm 3): the tokens of a cluster that were not kept as elites are
// averaged into one representative row.
//
// Two kernels on one stream:
//   merge_plan_kernel   one CTA per sample: gathers the non-elite tokens in token order and sorts them by label with
//                       a stable radix sort in shared memory, which lays every cluster's members out contiguously
//                       in ascending token order; the clusters that have members are numbered in ascending label
//                       order (ordered ballot/popc compaction of the run heads) and the member list goes to the
//                       workspace
//   merge_rows_kernel   one CTA per (merged row, sample, 512-byte slice of the hidden row): its four warps stream
//                       the members' row slices with 128-bit loads (member r goes to warp r mod 4) and the four
//                       fp32 partial sums are added in warp order, a fixed order (bit-reproducible).  Only rows
//                       that are averaged are read.
#include <cuda_bf16.h>

#include "internal.cuh"

namespace vitcop {
namespace {

constexpr int kPlanThreads = 1024;
constexpr int kPlanWarps = kPlanThreads / 32;
constexpr int kRowsThreads = 128;
constexpr int kPlanItems = VITCOP_MAX_VISUAL_TOKENS / kPlanThreads;   // rows of 32 entries a warp walks at most
constexpr int kDigitBits = 7, kDigits = 1 << kDigitBits;
static_assert(kDigits * kPlanWarps == 4 * kPlanThreads, "four counters per thread in the scan");
// The counter of (digit d, warp w) sits at w * kCntStride + d: the leaders of a row (one warp, distinct digits) and
// the four counters a thread scans (one digit, consecutive warps) both spread over the banks.
constexpr int kCntStride = kDigits + 2;
constexpr int kCntEntries = kPlanWarps * kCntStride;

// Every array of the planner is walked the same way: warp w owns the entries [w * 32 E, (w + 1) * 32 E), E =
// ceil(count / 1024), and takes them 32 at a time, lane by lane (coalesced, no bank conflicts, and entry order is
// (warp, row, lane) order, so that ballots and one scan over the 32 warp totals give stable positions).  The walks are
// rolled loops on purpose: the kernel runs once per call on a handful of SMs, so every instruction it executes is
// fetched cold, and a loop body fetched once beats sixteen unrolled copies.

// One walk of a warp over its items with a cursor per (digit, warp) in `cnt`: every item receives the cursor of its
// digit plus the number of items of the same digit in front of it in its row, and the cursor moves past the row's
// items.  With the cursors at zero the walk counts (dst null); with the cursors at their scanned values it writes the
// items to their sorted positions in dst.
__device__ __forceinline__ void digit_walk(const uint32_t* src, uint32_t* dst, int E, int m, int shift, uint16_t* cnt) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll 1
    for (int e = 0; e < E; ++e) {
        const int p = (warp * E + e) * 32 + lane;
        const bool valid = p < m;
        const uint32_t item = valid ? src[p] : 0u;
        const uint32_t d = (item >> shift) & (kDigits - 1);
        // the lanes of the row that hold the same digit: one ballot per bit
        const uint32_t vb = __ballot_sync(0xffffffffu, valid);
        uint32_t peers = valid ? vb : ~vb;
#pragma unroll
        for (int k = 0; k < kDigitBits; ++k) {
            const uint32_t bk = __ballot_sync(0xffffffffu, d >> k & 1u);
            peers &= (d >> k & 1u) ? bk : ~bk;
        }
        const int leader = __ffs(peers) - 1;
        uint32_t cur = 0;
        if (valid && lane == leader) {
            cur = cnt[warp * kCntStride + d];
            cnt[warp * kCntStride + d] = (uint16_t)(cur + __popc(peers));
        }
        cur = __shfl_sync(0xffffffffu, cur, leader);
        if (dst && valid) dst[cur + __popc(peers & ((1u << lane) - 1u))] = item;
        __syncwarp();                                      // the next row's leaders may be other lanes
    }
}

// Stable sort of m items (label << 16 | token index, in ascending token order on entry) by label: least significant
// digit first, seven bits at a time, from one buffer to the other and back.  Returns the buffer that holds the result.
// `cnt`: shared uint16_t [kCntEntries]; label_bits: bits of the largest label.
__device__ uint32_t* sort_by_label(uint32_t* a, uint32_t* b, int m, int label_bits, uint16_t* cnt, uint32_t* warp_sums) {
    const int t = threadIdx.x;
    const int E = (m + kPlanThreads - 1) / kPlanThreads;
    // this thread's four counters in scan order (digit by digit, inside a digit warp by warp)
    uint16_t* mine = cnt + (t % (kPlanWarps / 4)) * 4 * kCntStride + t / (kPlanWarps / 4);
#pragma unroll 1
    for (int shift = 16; shift < 16 + label_bits; shift += kDigitBits) {
        for (int c = t; c < kCntEntries; c += kPlanThreads) cnt[c] = 0;
        __syncthreads();
        digit_walk(a, nullptr, E, m, shift, cnt);
        __syncthreads();
        const uint32_t c0 = mine[0], c1 = mine[kCntStride], c2 = mine[2 * kCntStride], c3 = mine[3 * kCntStride];
        uint32_t total;
        const uint32_t b0 = block_exclusive_sum(c0 + c1 + c2 + c3, warp_sums, total);
        mine[0] = (uint16_t)b0;
        mine[kCntStride] = (uint16_t)(b0 + c0);
        mine[2 * kCntStride] = (uint16_t)(b0 + c0 + c1);
        mine[3 * kCntStride] = (uint16_t)(b0 + c0 + c1 + c2);
        __syncthreads();
        digit_walk(a, b, E, m, shift, cnt);
        __syncthreads();
        uint32_t* s = a;
        a = b;
        b = s;
    }
    return a;
}

__global__ void __launch_bounds__(kPlanThreads)
merge_plan_kernel(const int32_t* __restrict__ label, const uint8_t* __restrict__ keep_mask,
                  const int32_t* __restrict__ vis_len, int vis_len_uniform, int Nv_cap, int Mcap,
                  int32_t* __restrict__ merged_label, int32_t* __restrict__ merged_count,
                  int32_t* __restrict__ n_merged, uint16_t* __restrict__ members, int32_t* __restrict__ starts) {
    extern __shared__ __align__(16) uint32_t smem_items[];   // two item buffers of Nv_cap (rounded up to 4), then the counters
    __shared__ uint32_t warp_sums[32];
    grid_dependency_wait();
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t lt = (1u << lane) - 1u;
    int n = vis_len ? vis_len[b] : vis_len_uniform;
    n = max(0, min(n, Nv_cap));
    const int cap4 = (Nv_cap + 3) & ~3;
    uint32_t* buf0 = smem_items;
    uint32_t* buf1 = smem_items + cap4;
    uint16_t* cnt = reinterpret_cast<uint16_t*>(smem_items + 2 * cap4);
    label += (size_t)b * Nv_cap;
    keep_mask += (size_t)b * Nv_cap;
    merged_label += (size_t)b * Mcap;
    merged_count += (size_t)b * Mcap;
    members += (size_t)b * Nv_cap;
    starts += (size_t)b * Mcap;

    // ---- the non-elite tokens, in token order: count per warp, one scan, then place.  (Unrolled, unlike the walks
    //      over shared memory: all of a thread's global loads are in flight together.)
    uint32_t m;
    {
        const int E = (n + kPlanThreads - 1) / kPlanThreads;
        uint32_t it[kPlanItems], take = 0, mine = 0;
#pragma unroll
        for (int e = 0; e < kPlanItems; ++e) {
            const int i = (warp * E + e) * 32 + lane;
            if (e < E && i < n) {
                uint32_t lab = (uint32_t)label[i];
                if (lab >= (uint32_t)n) lab = (uint32_t)n - 1;     // out-of-range labels are clamped, never indexed
                it[e] = (lab << 16) | (uint32_t)i;
                if (!keep_mask[i]) take |= 1u << e;
            }
        }
#pragma unroll
        for (int e = 0; e < kPlanItems; ++e) mine += __popc(__ballot_sync(0xffffffffu, take >> e & 1u));
        uint32_t pos = warp_totals_scan(mine, warp_sums, m);
#pragma unroll
        for (int e = 0; e < kPlanItems; ++e) {
            const uint32_t bal = __ballot_sync(0xffffffffu, take >> e & 1u);
            if (take >> e & 1u) buf0[pos + __popc(bal & lt)] = it[e];
            pos += __popc(bal);
        }
    }
    __syncthreads();
    // ---- members of a cluster side by side, in ascending token order; clusters in ascending label order
    const uint32_t* items = sort_by_label(buf0, buf1, (int)m, n > 1 ? 32 - __clz(n - 1) : 0, cnt, warp_sums);

    // ---- run heads -> merged rows; run tails close them; the sorted indices are the member list
    const int E = ((int)m + kPlanThreads - 1) / kPlanThreads;
    uint32_t wh = 0, wt = 0;
#pragma unroll 1
    for (int e = 0; e < E; ++e) {
        const int p = (warp * E + e) * 32 + lane;
        bool head = false, tail = false;
        if (p < (int)m) {
            const uint32_t c = items[p], lab = c >> 16;
            head = p == 0 || (items[p - 1] >> 16) != lab;
            tail = p + 1 >= (int)m || (items[p + 1] >> 16) != lab;
            members[p] = (uint16_t)(c & 0xFFFFu);
        }
        wh += __popc(__ballot_sync(0xffffffffu, head));
        wt += __popc(__ballot_sync(0xffffffffu, tail));
    }
    // (two 16-bit counts in a word: neither can exceed 16384)
    uint32_t totals;
    const uint32_t before = warp_totals_scan(wh | (wt << 16), warp_sums, totals);
    uint32_t hs = before & 0xFFFFu, ts = before >> 16;
    const uint32_t heads = totals & 0xFFFFu;
#pragma unroll 1
    for (int e = 0; e < E; ++e) {
        const int p = (warp * E + e) * 32 + lane;
        bool head = false, tail = false;
        uint32_t lab = 0;
        if (p < (int)m) {
            lab = items[p] >> 16;
            head = p == 0 || (items[p - 1] >> 16) != lab;
            tail = p + 1 >= (int)m || (items[p + 1] >> 16) != lab;
        }
        const uint32_t hb = __ballot_sync(0xffffffffu, head), tb = __ballot_sync(0xffffffffu, tail);
        const uint32_t h = hs + __popc(hb & lt), t = ts + __popc(tb & lt);
        if (head && h < (uint32_t)Mcap) {
            merged_label[h] = (int32_t)lab;
            starts[h] = p;
        }
        if (tail && t < (uint32_t)Mcap) merged_count[t] = p;            // position of the run's last member for now
        hs += __popc(hb);
        ts += __popc(tb);
    }
    __syncthreads();
    for (int mm = tid; mm < min((int)heads, Mcap); mm += kPlanThreads) merged_count[mm] = merged_count[mm] - starts[mm] + 1;
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
    const int pl = tid & 31;                              // this thread finishes elements tid / 32, + G, .. of piece pl
    const int pcol = blockIdx.z * 32 + pl;
    if (pcol >= dh8) return;
#pragma unroll
    for (int k = tid >> 5; k < 8; k += G) {
        float sum = 0.f;
#pragma unroll
        for (int q = 0; q < G; ++q) sum += partial[q][pl][k];   // warp order: fixed
        sum = sum / (float)count;
        const size_t o = (((size_t)b * Mcap + m) * dh8 + pcol) * 8 + k;
        if (merged_f32) merged_f32[o] = sum;
        if (merged_bf16) static_cast<__nv_bfloat16*>(merged_bf16)[o] = __float2bfloat16_rn(sum);
    }
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
        const size_t smem = 2 * (size_t)((Nv_cap + 3) & ~3) * sizeof(uint32_t) + (size_t)kCntEntries * sizeof(uint16_t);
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
