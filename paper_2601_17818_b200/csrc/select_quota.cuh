// Cluster-quota selection (Eq. 5 / Algorithm 3 up to the elite set) as a CTA-wide device routine, called by
// select_quota_kernel (select.cu).
#pragma once

#include "block_sort.cuh"
#include "internal.cuh"

namespace vitcop {

constexpr int kSelThreads = 1024;
constexpr int kSelWarps = kSelThreads / 32;   // block_prefix_count (internal.cuh) is written for this size

// Ascending key order == the selection order: smaller scores first (or larger, when `largest`),
// -0 == +0, NaN after everything.
__device__ __forceinline__ uint32_t order_key(float s, int largest) {
    if (s != s) return 0xFFFFFFFFu;
    uint32_t u = __float_as_uint(s);
    if (u == 0x80000000u) u = 0u;
    const uint32_t asc = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
    return largest ? ~asc : asc;
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

// ------------------------------------------------------------------------------------------ per-cluster select
// Cluster-quota selection without a global sort, for up to kMaxSeg clusters.  Tokens get dense cluster ids, the
// clusters their sizes and quotas; then one of two searches finds, per cluster, the q_c smallest (score key, index)
// pairs:
//   rank   -- the tokens are scattered into per-cluster segments and every token counts the members of its own
//             segment that precede it: sum of |C_c|^2 comparisons, taken when that sum is a small multiple of n
//             (clusters of similar size, the usual outcome of Algorithm 2);
//   radix  -- every cluster runs its own radix select (4-bit digits) for its q_c-th smallest pair, all clusters at
//             once: one shared histogram row per cluster, one thread per cluster to pick the digit, O(n) work per
//             pass whatever the sizes.  Pairs are unique, so ties need no extra pass; a cluster stops as soon as a
//             whole histogram bin is wanted, the loop when all clusters have stopped.
constexpr int kMaxSeg = 1024;
constexpr int kSegTok = 16;                               // tokens per thread: VITCOP_MAX_VISUAL_TOKENS / kSelThreads
constexpr uint32_t kSegDone = 0xFFFFFFFFu;
constexpr int kRankWork = 64;                             // rank search when sum |C_c|^2 <= kRankWork * n ...
constexpr int kRankWorkLong = 16;                         // ... (long samples: a CTA's 1024 threads share all of it) ...
constexpr int kRankLongTokens = 8192;
constexpr int kRankMaxSize = 2048;                        // ... and no searched cluster is larger than this
constexpr int kRadixMinTokens = 4096;                     // below this a sort beats the radix passes (fewer barriers)

// Writes the tokens whose flag is set in keepf[0..n) to keep_idx in ascending order (every thread scans a run of
// consecutive tokens, one block-wide scan places the runs); returns their number.
__device__ __forceinline__ uint32_t emit_flags_ascending(int n, const uint8_t* keepf, int32_t* keep_idx,
                                                         int keep_stride, uint8_t* keep_mask, uint32_t* warp_sums) {
    const int per = (n + kSelThreads - 1) / kSelThreads;
    const int i0 = threadIdx.x * per;
    uint32_t cnt = 0;
    for (int j = 0; j < per; ++j) cnt += (i0 + j < n && keepf[i0 + j]) ? 1u : 0u;
    uint32_t total;
    uint32_t r = block_exclusive_sum(cnt, warp_sums, total);
    for (int j = 0; j < per; ++j) {
        const int i = i0 + j;
        if (i >= n) break;
        const bool f = keepf[i] != 0;
        if (f) {
            if (r < (uint32_t)keep_stride) keep_idx[r] = i;
            ++r;
        }
        if (keep_mask) keep_mask[i] = f ? 1 : 0;
    }
    return total;
}

// Shared-memory layout of select_quota_by_cluster for a sample of n tokens.
struct ClusterSelSmem {
    size_t off_thr, off_krem, off_quota, off_csize, off_offs, off_misc, off_id, off_keep, total;
    int n_al;
    __host__ __device__ explicit ClusterSelSmem(int n) {
        n_al = (n + 7) & ~7;
        size_t uni = (size_t)n_al * 8;                     // seg u64 [n_al]: tokens grouped by cluster   (rank)
        const size_t hist = (size_t)kMaxSeg * 16 * 4;      // hist u32 [copies][n_seg][16]              (radix)
        if (uni < hist) uni = hist;
        off_thr = uni;
        off_krem = off_thr + (size_t)kMaxSeg * 8;
        off_quota = off_krem + (size_t)kMaxSeg * 4;
        off_csize = off_quota + (size_t)kMaxSeg * 4;
        off_offs = off_csize + (size_t)kMaxSeg * 4;
        off_misc = off_offs + (size_t)kMaxSeg * 4;
        off_id = off_misc + 16;
        off_keep = off_id + (size_t)n_al * 2;
        total = off_keep + (size_t)n_al;
    }
};

// Returns false (having written nothing) when the sample has more than kMaxSeg clusters, or sizes that rule out
// the rank search on a sample too short for the radix search to pay: the caller then sorts.
__device__ __forceinline__ bool select_quota_by_cluster(const float* score, const int32_t* label, int n, int budget,
                                                        int32_t* keep_idx, int keep_stride, int32_t* n_keep_b,
                                                        uint8_t* keep_mask, int* status_word, uint8_t* smem,
                                                        uint32_t* warp_sums) {
    const ClusterSelSmem L(n);
    uint32_t* hist = reinterpret_cast<uint32_t*>(smem);
    unsigned long long* seg = reinterpret_cast<unsigned long long*>(smem);
    unsigned long long* thr = reinterpret_cast<unsigned long long*>(smem + L.off_thr);
    uint32_t* krem = reinterpret_cast<uint32_t*>(smem + L.off_krem);
    uint32_t* quota = reinterpret_cast<uint32_t*>(smem + L.off_quota);
    uint32_t* csize = reinterpret_cast<uint32_t*>(smem + L.off_csize);
    uint32_t* offs = reinterpret_cast<uint32_t*>(smem + L.off_offs);
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + L.off_misc);   // min key, max key, rank work, rank veto
    uint16_t* id_of = reinterpret_cast<uint16_t*>(smem + L.off_id);
    uint8_t* keepf = smem + L.off_keep;
    const int tid = threadIdx.x;

    // ---- dense cluster ids in ascending label order
    for (int i = tid; i < n; i += kSelThreads) id_of[i] = 0;
    if (tid < kMaxSeg) csize[tid] = 0;
    if (tid == 0) {
        misc[0] = 0xFFFFFFFFu;
        misc[1] = 0u;
        misc[2] = 0u;
        misc[3] = 0u;
    }
    __syncthreads();
    // per token: (cluster << 48) | (score key << 16) | low; low = slot inside the cluster first, then the index
    unsigned long long comp[kSegTok];
    uint32_t key_lo = 0xFFFFFFFFu, key_hi = 0u;
#pragma unroll
    for (int k = 0; k < kSegTok; ++k) {
        const int i = k * kSelThreads + tid;
        comp[k] = 0;
        if (i < n) {
            uint32_t lab = (uint32_t)label[i];
            if (lab >= (uint32_t)n) lab = (uint32_t)n - 1;          // out-of-range labels are clamped, never indexed
            id_of[lab] = 1;
            const uint32_t key = order_key(score[i], 0);
            key_lo = min(key_lo, key);
            key_hi = max(key_hi, key);
            comp[k] = ((unsigned long long)lab << 48) | ((unsigned long long)key << 16);
        }
    }
    key_lo = __reduce_min_sync(0xffffffffu, key_lo);
    key_hi = __reduce_max_sync(0xffffffffu, key_hi);
    if ((tid & 31) == 0) {
        atomicMin(&misc[0], key_lo);
        atomicMax(&misc[1], key_hi);
    }
    __syncthreads();
    const int per = (n + kSelThreads - 1) / kSelThreads;
    const int l0 = tid * per;
    uint32_t cnt = 0;
    for (int j = 0; j < per; ++j) cnt += (l0 + j < n && id_of[l0 + j]) ? 1u : 0u;
    uint32_t n_seg;
    uint32_t next_id = block_exclusive_sum(cnt, warp_sums, n_seg);
    if (n_seg > (uint32_t)kMaxSeg) return false;           // uniform over the CTA
    for (int j = 0; j < per; ++j)
        if (l0 + j < n && id_of[l0 + j]) id_of[l0 + j] = (uint16_t)next_id++;
    __syncthreads();

    // ---- cluster sizes (the atomic's return value is the token's slot inside its cluster) and quotas (Eq. 5)
#pragma unroll
    for (int k = 0; k < kSegTok; ++k) {
        if (k * kSelThreads + tid < n) {
            const uint32_t c = id_of[(uint32_t)(comp[k] >> 48)];
            const uint32_t slot = atomicAdd(&csize[c], 1u);
            comp[k] = (comp[k] & 0x0000FFFFFFFF0000ull) | ((unsigned long long)c << 48) | (unsigned long long)slot;
        }
    }
    __syncthreads();
    const long long b_elites = (long long)budget - (long long)n_seg;
    if (b_elites < 0) {
        if (tid == 0 && status_word) atomicMax(status_word, VITCOP_ERR_BUDGET);
        for (int i = tid; i < n; i += kSelThreads) keepf[i] = 0;
        __syncthreads();
        emit_flags_ascending(n, keepf, keep_idx, keep_stride, keep_mask, warp_sums);
        if (tid == 0) *n_keep_b = 0;
        return true;
    }
    {
        uint32_t size = 0, work = 0, veto = 0;
        if (tid < (int)n_seg) {
            size = csize[tid];
            const long long q = ((long long)size * b_elites) / (long long)n;
            quota[tid] = (uint32_t)q;
            const bool searched = q > 0 && q < (long long)size;      // none or all of a cluster: nothing to search
            krem[tid] = searched ? (uint32_t)q : kSegDone;
            if (searched) {
                veto = size > (uint32_t)kRankMaxSize ? 1u : 0u;
                work = veto ? 0u : size * size;
            }
        }
        work = __reduce_add_sync(0xffffffffu, work);
        veto = __reduce_or_sync(0xffffffffu, veto);
        if ((tid & 31) == 0 && (work | veto)) {
            atomicAdd(&misc[2], min(work, 0x0FFFFFFFu));             // 32 sizes of at most 2048: below 2^27
            atomicOr(&misc[3], veto);
        }
        uint32_t total;
        const uint32_t o = block_exclusive_sum(size, warp_sums, total);   // its barriers publish misc as well
        if (tid < (int)n_seg) offs[tid] = o;
    }
    const bool by_rank = misc[3] == 0 && (unsigned long long)misc[2] <=
                                             (unsigned long long)(n > kRankLongTokens ? kRankWorkLong : kRankWork) * (unsigned)n;
    const uint32_t range_lo = misc[0], range_hi = misc[1];
    if (!by_rank && n <= kRadixMinTokens) return false;    // uniform; nothing has been written yet
    __syncthreads();

    if (by_rank) {
        // ---- scatter into per-cluster segments; then the thread of segment position p ranks the token stored
        // there.  The lanes of a warp mostly sit in one cluster: equal trip counts and broadcast reads.
#pragma unroll
        for (int k = 0; k < kSegTok; ++k) {
            const int i = k * kSelThreads + tid;
            if (i < n) {
                const uint32_t c = (uint32_t)(comp[k] >> 48);
                seg[offs[c] + (uint32_t)(comp[k] & 0xFFFFull)] = (comp[k] & ~0xFFFFull) | (unsigned long long)i;
            }
        }
        __syncthreads();
        for (int p = tid; p < n; p += kSelThreads) {
            const unsigned long long mine = seg[p];
            const uint32_t c = (uint32_t)(mine >> 48);
            const uint32_t q = quota[c], size = csize[c];
            bool keep = q >= size;
            if (!keep && q > 0) {
                const unsigned long long* members = seg + offs[c];
                uint32_t before = 0;
                uint32_t m = 0;
                for (; m + 4 <= size; m += 4) {
                    const unsigned long long m0 = members[m], m1 = members[m + 1], m2 = members[m + 2],
                                             m3 = members[m + 3];
                    before += (m0 < mine ? 1u : 0u) + (m1 < mine ? 1u : 0u) + (m2 < mine ? 1u : 0u) +
                              (m3 < mine ? 1u : 0u);
                }
                for (; m < size; ++m) before += members[m] < mine ? 1u : 0u;
                keep = before < q;                        // same cluster bits: the order of (score key, index)
            }
            keepf[(uint32_t)(mine & 0xFFFFull)] = keep ? 1 : 0;
        }
    } else {
        // ---- per-cluster radix select of the quota-th smallest pair, 4 bits per pass from the top of the 48-bit
        // (score key, index) value.  The digits above the first bit in which two score keys differ are the same
        // for every token and are skipped.
#pragma unroll
        for (int k = 0; k < kSegTok; ++k)
            comp[k] = (comp[k] & ~0xFFFFull) | (unsigned long long)(k * kSelThreads + tid);
        const int same_bits = __clz((int)(range_lo ^ range_hi));                 // 32 when all scores are equal
        const int shift0 = ((47 - same_bits) / 4) * 4;
        const unsigned long long thr0 = (((unsigned long long)range_lo << 16) >> (shift0 + 4)) << (shift0 + 4);
        if (tid < (int)n_seg) thr[tid] = thr0;
        // few clusters: several copies of the histogram, one per group of warps, spread the shared-memory atomics
        int copies = 1;
        while (copies < 8 && (int)n_seg * 2 * copies <= kMaxSeg) copies <<= 1;
        uint32_t* my_hist = hist + (size_t)((tid >> 5) & (copies - 1)) * n_seg * 16;
        for (int shift = shift0; shift >= 0; shift -= 4) {
            for (int h = tid; h < (int)n_seg * 16 * copies; h += kSelThreads) hist[h] = 0;
            __syncthreads();
#pragma unroll
            for (int k = 0; k < kSegTok; ++k) {
                if (k * kSelThreads + tid < n) {
                    const uint32_t c = (uint32_t)(comp[k] >> 48);
                    if (krem[c] != kSegDone) {
                        const unsigned long long key = comp[k] & 0xFFFFFFFFFFFFull;
                        if ((key >> (shift + 4)) == (thr[c] >> (shift + 4)))
                            atomicAdd(&my_hist[c * 16 + (uint32_t)((key >> shift) & 15ull)], 1u);
                    }
                }
            }
            __syncthreads();
            int open_left = 0;
            if (tid < (int)n_seg) {
                const int c = tid;
                uint32_t kr = krem[c];
                if (kr != kSegDone) {
                    uint32_t cum = 0;
                    for (int dgt = 0; dgt < 16; ++dgt) {
                        uint32_t h = 0;
                        for (int r = 0; r < copies; ++r) h += hist[((size_t)r * n_seg + c) * 16 + dgt];
                        if (cum + h >= kr) {
                            unsigned long long t = thr[c] | ((unsigned long long)dgt << shift);
                            kr -= cum;
                            if (h == kr || shift == 0) {   // the whole bin is wanted: every pair up to its top is kept
                                t |= (1ull << shift) - 1ull;
                                krem[c] = kSegDone;
                            } else {
                                krem[c] = kr;
                                open_left = 1;
                            }
                            thr[c] = t;
                            break;
                        }
                        cum += h;
                    }
                }
            }
            if (!__syncthreads_or(open_left)) break;
        }
#pragma unroll
        for (int k = 0; k < kSegTok; ++k) {
            const int i = k * kSelThreads + tid;
            if (i < n) {
                const uint32_t c = (uint32_t)(comp[k] >> 48);
                const uint32_t q = quota[c];
                const bool keep = q >= csize[c] ? true : (q == 0 ? false : (comp[k] & 0xFFFFFFFFFFFFull) <= thr[c]);
                keepf[i] = keep ? 1 : 0;
            }
        }
    }
    __syncthreads();
    const uint32_t kept = emit_flags_ascending(n, keepf, keep_idx, keep_stride, keep_mask, warp_sums);
    if (tid == 0) *n_keep_b = (int32_t)kept;
    return true;
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

    if (select_quota_by_cluster(score, label, n, budget, keep_idx, keep_stride, n_keep + b, keep_mask, status_word,
                                reinterpret_cast<uint8_t*>(smem_u32), warp_sums))
        return;
    __syncthreads();
    // more clusters than the per-cluster searches handle, or a short sample with very uneven clusters: sort the
    // composites (label, score key, index)
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
    const size_t sort_bytes = (size_t)P * 8 + (size_t)cap * (2 + 2 + 1) + 16;
    const size_t seg_bytes = ClusterSelSmem(cap).total;
    return sort_bytes > seg_bytes ? sort_bytes : seg_bytes;
}

}  // namespace vitcop
