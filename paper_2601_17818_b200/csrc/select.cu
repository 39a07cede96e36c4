// Budgeted selection of visual tokens: one CTA per sequence, scores held in shared memory.
//
//  plain mode (Algorithm 1, Stage III / Stage I): exact k-th order statistic of the 32-bit
//    order-preserving score key by a 4-pass, 8-bit radix select; ties at the cut are resolved toward
//    the lower index by an ordered (ballot + popc) prefix count; the kept indices leave in ascending
//    order through a second ordered prefix count over the keep flags.
//  quota mode (Eq. 5 / Algorithm 3 up to the elite set): a bitonic sort of the 64-bit composite
//    (label, score key, index) groups the clusters and ranks their members; member r of cluster c is
//    kept iff r < q_c = (|C_c| * (budget - N_c)) / n.
#include "block_sort.cuh"
#include "internal.cuh"

namespace vitcop {
namespace {

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

// ------------------------------------------------------------------------------------------ plain
__global__ void __launch_bounds__(kSelThreads)
select_plain_kernel(const float* __restrict__ score, const int32_t* __restrict__ vis_len, int vis_len_uniform,
                    int Nv_cap, int largest, int budget, int32_t* __restrict__ keep_idx, int keep_stride,
                    int32_t* __restrict__ n_keep, uint8_t* __restrict__ keep_mask) {
    extern __shared__ __align__(16) uint32_t smem_u32[];
    uint32_t* keys = smem_u32;
    __shared__ uint32_t hist[256];
    __shared__ uint32_t warp_sums[kSelWarps];
    __shared__ uint32_t s_digit, s_krem, s_whole;

    grid_dependency_wait();
    const int b = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int n = vis_len ? vis_len[b] : vis_len_uniform;
    n = max(0, min(n, Nv_cap));
    const int k = max(0, min(budget, n));
    score += (int64_t)b * Nv_cap;
    keep_idx += (int64_t)b * keep_stride;
    if (keep_mask) keep_mask += (int64_t)b * Nv_cap;

    for (int i = tid; i < n; i += kSelThreads) keys[i] = order_key(score[i], largest);
    __syncthreads();

    uint32_t T = 0xFFFFFFFFu;   // cut key: keep key < T, plus `krem` of the key == T elements
    uint32_t krem = 0;
    if (k > 0 && k < n) {
        uint32_t prefix = 0;
        krem = (uint32_t)k;
        for (int pass = 0; pass < 4; ++pass) {
            const int shift = 24 - 8 * pass;
            const uint32_t hi_mask = pass == 0 ? 0u : (0xFFFFFFFFu << (shift + 8));
            if (tid < 256) hist[tid] = 0;
            __syncthreads();
            for (int base = 0; base < n; base += kSelThreads) {
                const int i = base + tid;
                int dig = -1;
                if (i < n) {
                    const uint32_t key = keys[i];
                    if ((key & hi_mask) == prefix) dig = (int)((key >> shift) & 255u);
                }
                const uint32_t peers = __match_any_sync(0xffffffffu, dig);
                if (dig >= 0 && lane == __ffs(peers) - 1) atomicAdd(&hist[dig], (uint32_t)__popc(peers));
            }
            __syncthreads();
            // inclusive scan of the 256 bins by the first 8 warps
            uint32_t c = tid < 256 ? hist[tid] : 0u;
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
                for (int w = 0; w < warp; ++w) basew += warp_sums[w];
                const uint32_t incl = basew + v, excl = incl - c;
                if (excl < krem && krem <= incl) {
                    s_digit = (uint32_t)tid;
                    s_krem = krem - excl;
                    s_whole = (c == krem - excl) ? 1u : 0u;         // the whole bin is wanted
                }
            }
            __syncthreads();
            prefix |= s_digit << shift;
            krem = s_krem;
            const bool whole = s_whole != 0;
            __syncthreads();
            if (whole) {
                // every key that shares the prefix found so far is kept: no need to resolve lower digits
                prefix |= (1u << shift) - 1u;
                krem = 0xFFFFFFFFu;
                break;
            }
        }
        T = prefix;
    }

    uint32_t kept;
    if (k == 0) {
        kept = emit_ascending(n, [](int) { return false; }, keep_idx, keep_stride, keep_mask, warp_sums);
    } else if (k >= n) {
        kept = emit_ascending(n, [](int) { return true; }, keep_idx, keep_stride, keep_mask, warp_sums);
    } else {
        // one sweep in index order: rank among the elements equal to the cut, then rank among the kept
        uint32_t eq_running = 0, keep_running = 0;
        for (int base = 0; base < n; base += kSelThreads) {
            const int i = base + tid;
            const uint32_t key = i < n ? keys[i] : 0xFFFFFFFFu;
            const bool eq = i < n && key == T;
            uint32_t eq_total, keep_total;
            const uint32_t eq_rank = eq_running + block_prefix_count(eq, warp_sums, eq_total);
            const bool f = i < n && (key < T || (eq && eq_rank < krem));
            const uint32_t r = keep_running + block_prefix_count(f, warp_sums, keep_total);
            if (f && r < (uint32_t)keep_stride) keep_idx[r] = i;
            if (keep_mask && i < n) keep_mask[i] = f ? 1 : 0;
            eq_running += eq_total;
            keep_running += keep_total;
        }
        kept = keep_running;
    }
    if (tid == 0) n_keep[b] = (int32_t)kept;
    grid_dependency_launch_dependents();
}

// Loads the composite keys (label, score key, index) of one sequence, padded with ~0 up to P, and sorts them.
template <int E>
__device__ void sort_composites(const float* __restrict__ score, const int32_t* __restrict__ label, int n, int T,
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
__global__ void __launch_bounds__(kSelThreads)
select_quota_kernel(const float* __restrict__ score, const int32_t* __restrict__ label,
                    const int32_t* __restrict__ vis_len, int vis_len_uniform, int Nv_cap, int P_cap, int budget,
                    int32_t* __restrict__ keep_idx, int keep_stride, int32_t* __restrict__ n_keep,
                    uint8_t* __restrict__ keep_mask, int* __restrict__ status_word) {
    extern __shared__ __align__(16) uint32_t smem_u32[];
    unsigned long long* comp = reinterpret_cast<unsigned long long*>(smem_u32);
    uint16_t* cstart = reinterpret_cast<uint16_t*>(comp + P_cap);
    uint16_t* csize = cstart + Nv_cap;
    uint8_t* keepf = reinterpret_cast<uint8_t*>(csize + Nv_cap);
    __shared__ uint32_t warp_sums[kSelWarps];

    grid_dependency_wait();
    const int b = blockIdx.x;
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
    grid_dependency_launch_dependents();
}

}  // namespace

int launch_select(const float* score, const int32_t* label, int B, const int32_t* vis_len, int vis_len_uniform,
                  int Nv_cap, int mode, int largest, int budget, int32_t* keep_idx, int keep_stride,
                  int32_t* n_keep, uint8_t* keep_mask, int* status_word, cudaStream_t stream, bool pdl) {
    if (B <= 0) return VITCOP_OK;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(B);
    cfg.blockDim = dim3(kSelThreads);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_allowed(pdl) ? 1 : 0;
    const int cap = Nv_cap > 0 ? Nv_cap : 1;
    if (mode == 0) {
        const size_t smem = (size_t)cap * sizeof(uint32_t);
        if (smem > 48 * 1024) {
            cudaError_t e = cudaFuncSetAttribute(select_plain_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 (int)smem);
            if (e != cudaSuccess) return record_cuda(e);
        }
        cfg.dynamicSmemBytes = smem;
        KernelTimeScope timed("select_plain_kernel", stream);
        return record_cuda(cudaLaunchKernelEx(&cfg, select_plain_kernel, score, vis_len, vis_len_uniform, Nv_cap,
                                              largest, budget, keep_idx, keep_stride, n_keep, keep_mask));
    }
    int P = 256;
    while (P < cap) P <<= 1;
    const size_t smem = (size_t)P * 8 + (size_t)cap * (2 + 2 + 1) + 16;
    if (smem > 48 * 1024) {
        cudaError_t e =
            cudaFuncSetAttribute(select_quota_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return record_cuda(e);
    }
    cfg.dynamicSmemBytes = smem;
    KernelTimeScope timed("select_quota_kernel", stream);
    return record_cuda(cudaLaunchKernelEx(&cfg, select_quota_kernel, score, label, vis_len, vis_len_uniform, Nv_cap,
                                          P, budget, keep_idx, keep_stride, n_keep, keep_mask, status_word));
}

}  // namespace vitcop
