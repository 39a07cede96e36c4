// Order-preserving compaction of hidden states and the K/V cache (bit-exact row gather).
//
// One CTA per (output row, sample).  The source position of the row comes from the ascending
// keep list; the CTA then moves the hidden row and the row of every K and V head with 128-bit
// loads that are all issued before the first store, so that each thread keeps several
// independent 16-byte requests in flight.  Dropped rows are never read.
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

// Copies `total` 16-byte pieces that sit in segments of `seg_len` pieces each (segment s starts at
// src + s * src_stride / dst + s * dst_stride): one hidden row is a single segment, the K (or V) rows of one
// token are H segments of d/8 pieces.  Four loads are issued before the first store.
__device__ __forceinline__ void copy_segments(const uint4* __restrict__ src, uint4* __restrict__ dst, int seg_len,
                                              int total, int64_t src_stride, int64_t dst_stride, int shift) {
    for (int q0 = threadIdx.x; q0 < total; q0 += 4 * kCompactThreads) {
        uint4 v[4];
        uint4* d[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int q = q0 + u * kCompactThreads;
            d[u] = nullptr;
            if (q < total) {
                const int sgm = shift >= 0 ? q >> shift : q / seg_len;
                const int e = q - sgm * seg_len;
                v[u] = ld_stream(src + sgm * src_stride + e);
                d[u] = dst + sgm * dst_stride + e;
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (d[u]) st_stream(d[u], v[u]);
    }
}

__global__ void __launch_bounds__(kCompactThreads)
compact_kernel(const uint4* __restrict__ hidden, const uint4* __restrict__ K, const uint4* __restrict__ V, int H, int N,
               int d8, int dh8, int d8_shift, const int32_t* __restrict__ seq_len, int vis_start,
               const int32_t* __restrict__ vis_len, int vis_len_uniform, const int32_t* __restrict__ keep_idx,
               int keep_stride, const int32_t* __restrict__ n_keep, uint4* __restrict__ hidden_out,
               uint4* __restrict__ K_out, uint4* __restrict__ V_out, int Ncap, int32_t* __restrict__ kept_pos,
               int32_t* __restrict__ out_len) {
    const int b = blockIdx.y;
    const int r = blockIdx.x;
    const int L = seq_len ? min(seq_len[b], N) : N;
    const int64_t head_in = (int64_t)N * d8, head_out = (int64_t)Ncap * d8;
    // A row in front of the visual span keeps its place whatever the selection turns out to be: it is copied
    // before this kernel waits for the selection, while the kernels that produce it are still running.  (The
    // tensors copied here are inputs of the whole call, complete before its first kernel started.)
    const bool prefix_row = r < min(vis_start, L) && r < Ncap;
    if (prefix_row) {
        if (hidden)
            copy_segments(hidden + ((int64_t)b * N + r) * dh8, hidden_out + ((int64_t)b * Ncap + r) * dh8, dh8, dh8, 0,
                          0, 31);
        if (K)
            copy_segments(K + ((int64_t)b * H * N + r) * d8, K_out + ((int64_t)b * H * Ncap + r) * d8, d8, H * d8,
                          head_in, head_out, d8_shift);
        if (V)
            copy_segments(V + ((int64_t)b * H * N + r) * d8, V_out + ((int64_t)b * H * Ncap + r) * d8, d8, H * d8,
                          head_in, head_out, d8_shift);
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

    if (hidden)
        copy_segments(hidden + ((int64_t)b * N + src_row) * dh8, hidden_out + ((int64_t)b * Ncap + r) * dh8, dh8, dh8, 0,
                      0, 31);
    if (K)
        copy_segments(K + ((int64_t)b * H * N + src_row) * d8, K_out + ((int64_t)b * H * Ncap + r) * d8, d8, H * d8,
                      head_in, head_out, d8_shift);
    if (V)
        copy_segments(V + ((int64_t)b * H * N + src_row) * d8, V_out + ((int64_t)b * H * Ncap + r) * d8, d8, H * d8,
                      head_in, head_out, d8_shift);
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
    cfg.gridDim = dim3(rows, B);
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
        static_cast<const uint4*>(V), H, N, d / 8, Dh / 8, d8_shift, seq_len, vis_start, vis_len, vis_len_uniform, keep_idx,
        keep_stride, n_keep, static_cast<uint4*>(hidden_out), static_cast<uint4*>(K_out), static_cast<uint4*>(V_out),
        Ncap, kept_pos, out_len));
}

}  // namespace vitcop
