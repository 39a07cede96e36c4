// Budgeted selection of visual tokens: one CTA per sequence, scores held in shared memory.
//
//  plain mode (Algorithm 1, Stage III / Stage I): exact k-th order statistic of the 32-bit
//    order-preserving score key by a 4-pass, 8-bit radix select; ties at the cut are resolved toward
//    the lower index by an ordered (ballot + popc) prefix count; the kept indices leave in ascending
//    order through a second ordered prefix count over the keep flags.
//  quota mode (Eq. 5 / Algorithm 3 up to the elite set): a bitonic sort of the 64-bit composite
//    (label, score key, index) groups the clusters and ranks their members; member r of cluster c is
//    kept iff r < q_c = (|C_c| * (budget - N_c)) / n.
#include "select_quota.cuh"

namespace vitcop {
namespace {

// ------------------------------------------------------------------------------------------ plain
__global__ void __launch_bounds__(kSelThreads)
select_plain_kernel(const float* __restrict__ score, const int32_t* __restrict__ vis_len, int vis_len_uniform,
                    int Nv_cap, int largest, int budget, int32_t* __restrict__ keep_idx, int keep_stride,
                    int32_t* __restrict__ n_keep, uint8_t* __restrict__ keep_mask) {
    extern __shared__ __align__(16) uint32_t smem_u32[];
    uint32_t* keys = smem_u32;
    __shared__ uint32_t hist[256];
    __shared__ uint32_t warp_sums[kSelWarps];
    __shared__ uint32_t s_digit, s_krem, s_whole, s_lo, s_hi;

    // The compaction that follows may start at once: it copies the rows that do not depend on the selection and
    // waits for this kernel to complete before it reads the kept indices.
    grid_dependency_launch_dependents();
    grid_dependency_wait();
    const int b = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int n = vis_len ? vis_len[b] : vis_len_uniform;
    n = max(0, min(n, Nv_cap));
    const int k = max(0, min(budget, n));
    score += (int64_t)b * Nv_cap;
    keep_idx += (int64_t)b * keep_stride;
    if (keep_mask) keep_mask += (int64_t)b * Nv_cap;

    if (tid == 0) { s_lo = 0xFFFFFFFFu; s_hi = 0u; }
    __syncthreads();
    {
        uint32_t lo = 0xFFFFFFFFu, hi = 0u;
        for (int i = tid; i < n; i += kSelThreads) {
            const uint32_t key = order_key(score[i], largest);
            keys[i] = key;
            lo = min(lo, key);
            hi = max(hi, key);
        }
        lo = __reduce_min_sync(0xffffffffu, lo);
        hi = __reduce_max_sync(0xffffffffu, hi);
        if (lane == 0 && lo <= hi) {
            atomicMin(&s_lo, lo);
            atomicMax(&s_hi, hi);
        }
    }
    __syncthreads();

    uint32_t T = 0xFFFFFFFFu;   // cut key: keep key < T, plus `krem` of the key == T elements
    uint32_t krem = 0;
    if (k > 0 && k < n) {
        // The keys of a sample share their leading bits (norms of one layer lie within a few octaves): the passes
        // start at the highest bit in which two keys differ, eight bits at a time down to bit 0.
        const int top = 32 - __clz(s_lo ^ s_hi);            // bits [top, 32) are common to all keys; 0: all keys equal
        uint32_t prefix = top >= 32 ? 0u : (s_hi >> top) << top;
        krem = (uint32_t)k;
        for (int hi_bit = top; hi_bit > 0; hi_bit -= 8) {
            const int shift = hi_bit > 8 ? hi_bit - 8 : 0;
            const uint32_t digit_mask = (1u << (hi_bit - shift)) - 1u;
            const uint32_t hi_mask = hi_bit >= 32 ? 0u : (0xFFFFFFFFu << hi_bit);
            if (tid < 256) hist[tid] = 0;
            __syncthreads();
            for (int base = 0; base < n; base += kSelThreads) {
                const int i = base + tid;
                int dig = -1;
                if (i < n) {
                    const uint32_t key = keys[i];
                    if ((key & hi_mask) == prefix) dig = (int)((key >> shift) & digit_mask);
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
        // Ranks in index order -- first among the elements equal to the cut, then among the kept -- with two scans for
        // the whole sample: warp w owns the tokens [w * 32 E, (w + 1) * 32 E) and takes them 32 at a time, so that a
        // ballot gives the rank inside a row and one scan over the 32 warp totals the rest.
        const int E = (n + kSelThreads - 1) / kSelThreads;
        const uint32_t lt = (1u << lane) - 1u;
        uint32_t weq = 0;
        for (int e = 0; e < E; ++e) {
            const int i = (warp * E + e) * 32 + lane;
            weq += __popc(__ballot_sync(0xffffffffu, i < n && keys[i] == T));
        }
        uint32_t total;
        uint32_t eq_run = warp_totals_scan(weq, warp_sums, total);
        uint32_t fbits = 0, wkeep = 0;                     // bit e: this thread's token of row e is kept
        for (int e = 0; e < E; ++e) {
            const int i = (warp * E + e) * 32 + lane;
            const uint32_t key = i < n ? keys[i] : 0xFFFFFFFFu;
            const bool eq = i < n && key == T;
            const uint32_t bal = __ballot_sync(0xffffffffu, eq);
            const bool f = i < n && (key < T || (eq && eq_run + __popc(bal & lt) < krem));
            eq_run += __popc(bal);
            fbits |= (uint32_t)f << e;
            wkeep += __popc(__ballot_sync(0xffffffffu, f));
        }
        uint32_t r = warp_totals_scan(wkeep, warp_sums, total);
        for (int e = 0; e < E; ++e) {
            const int i = (warp * E + e) * 32 + lane;
            const bool f = (fbits >> e & 1u) != 0;
            const uint32_t bal = __ballot_sync(0xffffffffu, f);
            const uint32_t at = r + __popc(bal & lt);
            if (f && at < (uint32_t)keep_stride) keep_idx[at] = i;
            if (keep_mask && i < n) keep_mask[i] = f ? 1 : 0;
            r += __popc(bal);
        }
        kept = total;
    }
    if (tid == 0) n_keep[b] = (int32_t)kept;
}

// ------------------------------------------------------------------------------------------ quota
__global__ void __launch_bounds__(kSelThreads)
select_quota_kernel(const float* __restrict__ score, const int32_t* __restrict__ label,
                    const int32_t* __restrict__ vis_len, int vis_len_uniform, int Nv_cap, int P_cap, int budget,
                    int32_t* __restrict__ keep_idx, int keep_stride, int32_t* __restrict__ n_keep,
                    uint8_t* __restrict__ keep_mask, int* __restrict__ status_word) {
    grid_dependency_launch_dependents();                  // see select_plain_kernel
    grid_dependency_wait();
    select_quota_body(score, label, vis_len, vis_len_uniform, Nv_cap, P_cap, budget, keep_idx, keep_stride, n_keep,
                      keep_mask, status_word, blockIdx.x);
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
    int P = 0;
    const size_t smem = select_quota_smem(Nv_cap, &P);
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
