// Per-token arithmetic of the K-norm (Eq. 4), shared by the stand-alone kernel (knorm.cu) and the resident Gram
// kernel (gram.cu), whose epilogue warps run it while they wait for the tensor cores.
#pragma once

#include "internal.cuh"

namespace vitcop {

__device__ __forceinline__ uint4 knorm_ld_stream(const uint4* p) {
    uint4 v;
    asm("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ void knorm_sq_acc(const uint4& v, float& a0, float& a1) {
    float x;
    x = bf16lo(v.x); a0 = fmaf(x, x, a0);
    x = bf16hi(v.x); a1 = fmaf(x, x, a1);
    x = bf16lo(v.y); a0 = fmaf(x, x, a0);
    x = bf16hi(v.y); a1 = fmaf(x, x, a1);
    x = bf16lo(v.z); a0 = fmaf(x, x, a0);
    x = bf16hi(v.z); a1 = fmaf(x, x, a1);
    x = bf16lo(v.w); a0 = fmaf(x, x, a0);
    x = bf16hi(v.w); a1 = fmaf(x, x, a1);
}

// Sum of squares of the 16-byte pieces sub, sub + LPR, ... of one token's K rows over all H heads (`base` points at
// the token's row in head 0; strides in 16-byte units).  The loads of head batch k + 1 are issued before the
// squares of batch k are accumulated, so that a thread always has UNROLL requests in flight.
template <int LPR, int UNROLL>
__device__ __forceinline__ float knorm_token_partial(const uint4* base, int H, int d8, int64_t sh, int sub) {
    float a0 = 0.f, a1 = 0.f;
    for (int c = sub; c < d8; c += LPR) {
        const uint4* p = base + c;
        const int full = H / UNROLL * UNROLL;
        if (full > 0) {
            uint4 cur[UNROLL], nxt[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) cur[u] = knorm_ld_stream(p + (int64_t)u * sh);
            for (int h = UNROLL; h < full; h += UNROLL) {
#pragma unroll
                for (int u = 0; u < UNROLL; ++u) nxt[u] = knorm_ld_stream(p + (int64_t)(h + u) * sh);
#pragma unroll
                for (int u = 0; u < UNROLL; ++u) knorm_sq_acc(cur[u], a0, a1);
#pragma unroll
                for (int u = 0; u < UNROLL; ++u) cur[u] = nxt[u];
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) knorm_sq_acc(cur[u], a0, a1);
        }
        for (int h = full; h < H; ++h) {
            const uint4 v = knorm_ld_stream(p + (int64_t)h * sh);
            knorm_sq_acc(v, a0, a1);
        }
    }
    return a0 + a1;
}

}  // namespace vitcop
