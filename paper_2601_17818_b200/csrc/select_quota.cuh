// Cluster-quota selection (Eq. 5 / Algorithm 3 up to the elite set) as a CTA-wide device routine, called by
// select_quota_kernel (select.cu).
#pragma once

#include "block_sort.cuh"
#include "internal.cuh"

namespace vitcop {

constexpr int kSelThreads = 1024;
constexpr int kSelWarps = kSelThreads / 32;

// Ascending key order == the selection order: smaller scores first (or larger, when `largest`),
// -0 == +0, NaN after everything.
__device__ __forceinline__ uint32_t order_key(float s, int largest) {
    if (s != s) return 0xFFFFFFFFu;
    uint32_t u = __float_as_uint(s);
    if (u == 0x80000000u) u = 0u;
    const uint32_t asc = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
    return largest ? ~asc : asc;
}

// Exclusive prefix count of `flag` over the CTA in thread order; `total` receives the CTA-wide count.
// Must be called by all threads.  warp_sums: shared uint32_t[kSelWarps].
__device__ __forceinline__ uint32_t block_prefix_count(bool flag, uint32_t* warp_sums, uint32_t& total) {
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

// Writes keep flags (already decided per element) out in ascending index order.
// flag_of(i) -> bool for i < n.  All threads call.
template <typename F>
__device__ __forceinline__ uint32_t emit_ascending(int n, F flag_of, int32_t* keep_idx, int keep_stride,
                                                   uint8_t* keep_mask, uint32_t* warp_sums) {
    uint32_t running = 0;
    for (int base = 0; base < n; base += kSelThreads) {
        const int i = base + threadIdx.x;
        const bool f = i < n && flag_of(i);
        uint32_t total;
        const uint32_t r = running + block_prefix_count(f, warp_sums, total);
        if (f && r < (uint32_t)keep_stride) keep_idx[r] = i;
        if (keep_mask && i < n) keep_mask[i] = f ? 1 : 0;
        running += total;
    }
    return running;
}

// Loads the composite keys (label, score key, index) of one sequence, padded with ~0 up to P, and sorts them.
template <int E>
__device__ void sort_composites(const float* score, const int32_t* label, int n, int T,
                                unsigned long long* comp) {
    unsigned long long r[E];
    const int t = threadIdx.x;
#pragma unroll
    for (int e = 0; e < E; ++e) {
        const int i = t * E + e;
        unsigned long long c = ~0ull;
        if (t < T && i < n) {
            uint32_t lab = (uint32_t)label[i];
            if (lab >= (uint32_t)n) lab = (uint32_t)n - 1;          // out-of-range labels are clamped, never indexed
            c = ((unsigned long long)lab << 48) | ((unsigned long long)order_key(score[i], 0) << 16) |
                (unsigned long long)i;
        }
        r[e] = c;
    }
    block_bitonic_sort<E>(r, comp, T);
}

// ------------------------------------------------------------------------------------------ quota
// Shared memory: comp[P] (uint64), cstart[n] and csize[n] (uint16, indexed by label value), keep[n] (uint8).
// Cluster-quota selection of sample b by the whole CTA (kSelThreads threads); uses the dynamic shared memory.
__device__ __forceinline__ void select_quota_body(const float* score, const int32_t* label,
                                                  const int32_t* __restrict__ vis_len, int vis_len_uniform,
                                                  int Nv_cap, int P_cap, int budget, int32_t* __restrict__ keep_idx,
                                                  int keep_stride, int32_t* __restrict__ n_keep,
                                                  uint8_t* __restrict__ keep_mask, int* __restrict__ status_word,
                                                  int b) {
    extern __shared__ __align__(16) uint32_t smem_u32[];
    unsigned long long* comp = reinterpret_cast<unsigned long long*>(smem_u32);
    uint16_t* cstart = reinterpret_cast<uint16_t*>(comp + P_cap);
    uint16_t* csize = cstart + Nv_cap;
    uint8_t* keepf = reinterpret_cast<uint8_t*>(csize + Nv_cap);
    __shared__ uint32_t warp_sums[kSelWarps];

    const int tid = threadIdx.x;
    int n = vis_len ? vis_len[b] : vis_len_uniform;
    n = max(0, min(n, Nv_cap));
    score += (int64_t)b * Nv_cap;
    label += (int64_t)b * Nv_cap;
    keep_idx += (int64_t)b * keep_stride;
    if (keep_mask) keep_mask += (int64_t)b * Nv_cap;

    int P = 256;                                          // at least one warp of 8 keys per thread
    while (P < n) P <<= 1;
    for (int i = tid; i < n; i += kSelThreads) keepf[i] = 0;
    if (P <= 8 * kSelThreads) sort_composites<8>(score, label, n, P / 8, comp);
    else sort_composites<16>(score, label, n, P / 16, comp);

    // cluster heads / tails in the sorted order
    uint32_t heads_here = 0;
    for (int p = tid; p < n; p += kSelThreads) {
        const uint32_t lab = (uint32_t)(comp[p] >> 48);
        if (p == 0 || (uint32_t)(comp[p - 1] >> 48) != lab) {
            cstart[lab] = (uint16_t)p;
            ++heads_here;
        }
    }
    __syncthreads();
    for (int p = tid; p < n; p += kSelThreads) {
        const uint32_t lab = (uint32_t)(comp[p] >> 48);
        if (p == n - 1 || (uint32_t)(comp[p + 1] >> 48) != lab) csize[lab] = (uint16_t)(p - cstart[lab]);  // size - 1
    }
    // N_c = number of heads
    uint32_t nc = heads_here;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) nc += __shfl_xor_sync(0xffffffffu, nc, off);
    if ((tid & 31) == 0) warp_sums[tid >> 5] = nc;
    __syncthreads();
    nc = 0;
    for (int w = 0; w < kSelWarps; ++w) nc += warp_sums[w];
    __syncthreads();

    const long long b_elites = (long long)budget - (long long)nc;
    if (b_elites < 0) {
        if (tid == 0 && status_word) atomicMax(status_word, VITCOP_ERR_BUDGET);
    } else {
        for (int p = tid; p < n; p += kSelThreads) {
            const unsigned long long c = comp[p];
            const uint32_t lab = (uint32_t)(c >> 48);
            const long long size_c = (long long)csize[lab] + 1;
            const long long q = (size_c * b_elites) / (long long)n;
            if ((long long)(p - (int)cstart[lab]) < q) keepf[(uint32_t)(c & 0xFFFFull)] = 1;
        }
    }
    __syncthreads();
    const uint32_t kept =
        emit_ascending(n, [&](int i) { return keepf[i] != 0; }, keep_idx, keep_stride, keep_mask, warp_sums);
    if (tid == 0) n_keep[b] = (int32_t)kept;
}


// Dynamic shared memory select_quota_body needs for a span capacity of Nv_cap tokens; *P_cap receives the padded key count.
inline size_t select_quota_smem(int Nv_cap, int* P_cap) {
    const int cap = Nv_cap > 0 ? Nv_cap : 1;
    int P = 256;
    while (P < cap) P <<= 1;
    *P_cap = P;
    return (size_t)P * 8 + (size_t)cap * (2 + 2 + 1) + 16;
}

}  // namespace vitcop
