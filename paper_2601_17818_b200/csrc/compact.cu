// Order-preserving compaction of hidden states and the K/V cache (bit-exact row gather).
//
// One CTA per (output row, sample).  The source position of the row comes from the ascending
// keep list; the CTA then moves the hidden row and the row of every K and V head with 128-bit
// loads, up to eight of them issued before the first store and taken from all three tensors alike, so that
// each thread keeps several independent 16-byte requests in flight.  Dropped rows are never read.
#include "internal.cuh"

namespace vitcop {
namespace {

constexpr int kCompactThreads = 256;

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream(uint4* p, const uint4& v) {
    asm volatile("st.global.L1::no_allocate.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z),
                 "r"(v.w)
                 : "memory");
}

// Moves one token: its hidden row (dh8 pieces of 16 bytes, one run) and its row in each of the H heads of K and of
// V (d8 pieces per head, heads head_in / head_out pieces apart).  The pieces of all three tensors form one index
// space, so that a thread has up to eight loads from any of them in flight before its first store: the row costs
// one round trip to memory, not one per tensor.  Null tensors are skipped.
__device__ __forceinline__ void copy_token(const uint4* __restrict__ hid_src, uint4* __restrict__ hid_dst, int dh8,
                                           const uint4* __restrict__ k_src, uint4* __restrict__ k_dst,
                                           const uint4* __restrict__ v_src, uint4* __restrict__ v_dst, int H, int d8,
                                           int d8_shift, int64_t head_in, int64_t head_out) {
    const int n_hid = hid_src ? dh8 : 0;
    const int n_kv = H * d8;
    const int n_k = k_src ? n_kv : 0;
    const int total = n_hid + n_k + (v_src ? n_kv : 0);
    constexpr int kInFlight = 8;
    for (int q0 = threadIdx.x; q0 < total; q0 += kInFlight * kCompactThreads) {
        uint4 v[kInFlight];
        uint4* d[kInFlight];
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) {
            int q = q0 + u * kCompactThreads;
            d[u] = nullptr;
            if (q < total) {
                if (q < n_hid) {
                    v[u] = ld_stream(hid_src + q);
                    d[u] = hid_dst + q;
                } else {
                    q -= n_hid;
                    const bool is_k = q < n_k;
                    if (!is_k) q -= n_k;
                    const int head = d8_shift >= 0 ? q >> d8_shift : q / d8;
                    const int e = q - head * d8;
                    v[u] = ld_stream((is_k ? k_src : v_src) + head * head_in + e);
                    d[u] = (is_k ? k_dst : v_dst) + head * head_out + e;
                }
            }
        }
#pragma unroll
        for (int u = 0; u < kInFlight; ++u)
            if (d[u]) st_stream(d[u], v[u]);
    }
}

__global__ void __launch_bounds__(kCompactThreads, 4)
compact_kernel(const uint4* __restrict__ hidden, const uint4* __restrict__ K, const uint4* __restrict__ V, int B, int H, int N,
               int d8, int dh8, int d8_shift, const int32_t* __restrict__ seq_len, int vis_start,
               const int32_t* __restrict__ vis_len, int vis_len_uniform, const int32_t* __restrict__ keep_idx,
               int keep_stride, const int32_t* __restrict__ n_keep, uint4* __restrict__ hidden_out,
               uint4* __restrict__ K_out, uint4* __restrict__ V_out, int Ncap, int32_t* __restrict__ kept_pos,
               int32_t* __restrict__ out_len) {
    // CTAs are handed out sample by sample within a row: all the rows in front of the visual span, which need not
    // wait for the selection, start before the rows that do
    const int r = (int)(blockIdx.x / (unsigned)B);
    const int b = (int)(blockIdx.x - (unsigned)r * (unsigned)B);
    const int L = seq_len ? min(seq_len[b], N) : N;
    const int64_t head_in = (int64_t)N * d8, head_out = (int64_t)Ncap * d8;
    // A row in front of the visual span keeps its place whatever the selection turns out to be: it is copied
    // before this kernel waits for the selection, while the kernels that produce it are still running.  (The
    // tensors copied here are inputs of the whole call, complete before its first kernel started.)
    const bool prefix_row = r < min(vis_start, L) && r < Ncap;
    if (prefix_row) {
        copy_token(hidden ? hidden + ((int64_t)b * N + r) * dh8 : nullptr, hidden_out + ((int64_t)b * Ncap + r) * dh8, dh8,
                   K ? K + ((int64_t)b * H * N + r) * d8 : nullptr, K_out + ((int64_t)b * H * Ncap + r) * d8,
                   V ? V + ((int64_t)b * H * N + r) * d8 : nullptr, V_out + ((int64_t)b * H * Ncap + r) * d8, H, d8,
                   d8_shift, head_in, head_out);
        if (kept_pos && threadIdx.x == 0) kept_pos[(int64_t)b * Ncap + r] = r;
        if (r != 0) return;                                // row 0 still reports the sample's new length
    }
    grid_dependency_wait();
    int nv = vis_len ? vis_len[b] : vis_len_uniform;
    nv = max(0, min(nv, L - vis_start));
    const int nk = max(0, min(n_keep[b], nv));
    const int olen = L - nv + nk;
    if (r == 0 && threadIdx.x == 0) out_len[b] = olen;
    if (r >= Ncap || prefix_row) return;
    if (r >= olen) {
        if (kept_pos && threadIdx.x == 0) kept_pos[(int64_t)b * Ncap + r] = -1;
        return;
    }
    int src_row;
    if (r < vis_start) src_row = r;
    else if (r < vis_start + nk) {
        int ki = keep_idx[(int64_t)b * keep_stride + (r - vis_start)];
        ki = max(0, min(ki, nv - 1));                     // a corrupt index can never leave the span
        src_row = vis_start + ki;
    } else src_row = r - nk + nv;
    if (kept_pos && threadIdx.x == 0) kept_pos[(int64_t)b * Ncap + r] = src_row;

    copy_token(hidden ? hidden + ((int64_t)b * N + src_row) * dh8 : nullptr, hidden_out + ((int64_t)b * Ncap + r) * dh8,
               dh8, K ? K + ((int64_t)b * H * N + src_row) * d8 : nullptr, K_out + ((int64_t)b * H * Ncap + r) * d8,
               V ? V + ((int64_t)b * H * N + src_row) * d8 : nullptr, V_out + ((int64_t)b * H * Ncap + r) * d8, H, d8,
               d8_shift, head_in, head_out);
}

}  // namespace

int launch_compact(const void* hidden, const void* K, const void* V, int B, int H, int N, int d, int Dh,
                   const int32_t* seq_len, int vis_start, const int32_t* vis_len, int vis_len_uniform,
                   const int32_t* keep_idx, int keep_stride, const int32_t* n_keep, void* hidden_out, void* K_out,
                   void* V_out, int Ncap, int32_t* kept_pos, int32_t* out_len, cudaStream_t stream, bool pdl) {
    if (B <= 0) return VITCOP_OK;
    const int d8 = d / 8;
    int d8_shift = -1;                                    // log2(d / 8) when that is a power of two
    if (d8 > 0 && (d8 & (d8 - 1)) == 0)
        for (d8_shift = 0; (1 << d8_shift) < d8; ++d8_shift) {}
    cudaLaunchConfig_t cfg = {};
    // rows past min(N, Ncap) cannot exist; one extra CTA row keeps out_len written when Ncap == 0
    const int rows = Ncap > 0 ? Ncap : 1;
    cfg.gridDim = dim3((unsigned)((long long)B * rows));
    cfg.blockDim = dim3(kCompactThreads);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_allowed(pdl) ? 1 : 0;
    KernelTimeScope timed("compact_kernel", stream);
    return record_cuda(cudaLaunchKernelEx(
        &cfg, compact_kernel, static_cast<const uint4*>(hidden), static_cast<const uint4*>(K),
        static_cast<const uint4*>(V), B, H, N, d / 8, Dh / 8, d8_shift, seq_len, vis_start, vis_len, vis_len_uniform, keep_idx,
        keep_stride, n_keep, static_cast<uint4*>(hidden_out), static_cast<uint4*>(K_out), static_cast<uint4*>(V_out),
        Ncap, kept_pos, out_len));
}

}  // namespace vitcop
