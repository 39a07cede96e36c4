// Internal declarations shared by the translation units of libvitcop (not part of the public ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "vitcop.h"

namespace vitcop {

// Device status word lives in the first 256 bytes of every workspace.
constexpr size_t kStatusBytes = 256;

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Records the first failing CUDA runtime error of the calling thread.
int record_cuda(cudaError_t e);

// Diagnostic per-kernel timing (vitcop_kernel_timing_begin / _end).  While it is on, a KernelTimeScope
// around a launch records one CUDA event before and one after the kernel on its stream, and launchers
// drop the programmatic-dependent-launch attribute so that consecutive kernels do not overlap.
bool kernel_timing_on();
struct KernelTimeScope {
    KernelTimeScope(const char* name, cudaStream_t stream);
    ~KernelTimeScope();
    KernelTimeScope(const KernelTimeScope&) = delete;
    KernelTimeScope& operator=(const KernelTimeScope&) = delete;
private:
    int slot_;
    cudaStream_t stream_;
};
inline bool pdl_allowed(bool requested) { return requested && !kernel_timing_on(); }

// ---- launchers (enqueue on `stream`, return VITCOP_OK or VITCOP_ERR_CUDA) -------------------------
int launch_knorm(const void* K, int B, int H, int d, int64_t stride_b, int64_t stride_h, int64_t stride_n,
                 int vis_start, const int32_t* vis_len, int vis_len_uniform, float* score, int Nv_cap,
                 cudaStream_t stream, bool late_wait = false, bool* launched = nullptr);
// (`launched`, when given, tells whether a kernel was enqueued at all: an empty span needs none.)

// K-norm to be enqueued in the middle of the filter's kernel chain (vitcop_collaborative_step): it does not depend
// on the filter, so it runs beside the filter's sweep.
struct KnormJob {
    const void* K;
    int B, H, N, d, vis_start, Nv;
    float* score;
};

int launch_select(const float* score, const int32_t* label, int B, const int32_t* vis_len, int vis_len_uniform,
                  int Nv_cap, int mode, int largest, int budget, int32_t* keep_idx, int keep_stride,
                  int32_t* n_keep, uint8_t* keep_mask, int* status_word, cudaStream_t stream, bool pdl);

int launch_compact(const void* hidden, const void* K, const void* V, int B, int H, int N, int d, int Dh,
                   const int32_t* seq_len, int vis_start, const int32_t* vis_len, int vis_len_uniform,
                   const int32_t* keep_idx, int keep_stride, const int32_t* n_keep, void* hidden_out, void* K_out,
                   void* V_out, int Ncap, int32_t* kept_pos, int32_t* out_len, cudaStream_t stream, bool pdl);

size_t filter_workspace_bytes(int B, int n, int D);
// Leading bytes of the filter workspace that must be zero when launch_filter starts (status block and flags).
size_t filter_zeroed_bytes(int B, int n);
size_t similarity_workspace_bytes(int B, int n, int D);
int launch_filter(const void* feat, const float* pos, int B, int n, int D, const vitcop_filter_params& p,
                  int n_centers, int32_t* label, int32_t* n_clusters, float* rho, float* delta2, int32_t* parent,
                  void* workspace, cudaStream_t stream, const KnormJob* knorm = nullptr);
int launch_similarity_rows(const void* feat, int B, int n, int D, int metric, int row_begin, int row_end,
                           float* out, void* workspace, cudaStream_t stream);

int launch_merge(const void* hidden, int B, int N, int Dh, int vis_start, const int32_t* vis_len, int vis_len_uniform,
                 int Nv_cap, const int32_t* label, const uint8_t* keep_mask, void* merged_bf16, float* merged_f32,
                 int32_t* merged_label, int32_t* merged_count, int32_t* n_merged, int Mcap, void* workspace,
                 cudaStream_t stream);
size_t merge_workspace_bytes(int B, int Nv_cap, int Mcap);

size_t kproj_workspace_bytes(int B, int N, int H, int d);
int launch_kproj_knorm(const void* hidden, const void* W, int B, int N, int Dh, int H, int d, const float* cos_tab,
                       const float* sin_tab, const int32_t* position, int n_pos, void* K_out, int vis_start, int Nv,
                       float* score, void* workspace, cudaStream_t stream);

size_t saliency_workspace_bytes(int B, int H, int M);
int launch_cls_saliency(const void* q, const void* K, int B, int H, int M, int d, float scale, float* saliency,
                        float* cls_self, void* workspace, cudaStream_t stream);

// ---- small device helpers ---------------------------------------------------------------------------
#ifdef __CUDACC__
__device__ __forceinline__ float bf16lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }

// Programmatic dependent launch: wait until the preceding kernel on the stream has completed
// (no-op when the kernel was not launched with the PDL attribute).
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_launch_dependents() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// Exclusive prefix count of `flag` over a CTA of 1024 threads, in thread order; `total` receives the CTA-wide
// count.  Must be called by all threads.  warp_sums: shared uint32_t[32].
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

// Exclusive prefix sum of one value per thread over a CTA of 1024 threads, in thread order; `total` receives the CTA-wide sum.
__device__ __forceinline__ uint32_t block_exclusive_sum(uint32_t v, uint32_t* warp_sums, uint32_t& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t incl = v;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += t;
    }
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    uint32_t w = warp_sums[lane];
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, w, off);
        if (lane >= off) w += t;
    }
    total = __shfl_sync(0xffffffffu, w, 31);
    const uint32_t base = warp == 0 ? 0u : __shfl_sync(0xffffffffu, w, warp - 1);
    __syncthreads();
    return base + incl - v;
}

// Exclusive prefix of one value per warp (uniform inside the warp) over the 32 warps of a CTA of 1024 threads; `total` = the sum.
__device__ __forceinline__ uint32_t warp_totals_scan(uint32_t warp_total, uint32_t* warp_sums, uint32_t& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) warp_sums[warp] = warp_total;
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
    return warp == 0 ? 0u : base;
}

#endif

}  // namespace vitcop
