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

// a0 += (low halves)^2, a1 += (high halves)^2 of the four bf16 pairs, pair by pair: the two accumulators advance
// together as one fp32x2 fused multiply-add per pair (each half rounded like the scalar instruction).
__device__ __forceinline__ void knorm_sq_acc(const uint4& v, float& a0, float& a1) {
    unsigned long long acc;
    asm("mov.b64 %0, {%1, %2};" : "=l"(acc) : "f"(a0), "f"(a1));
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        unsigned long long x;
        asm("mov.b64 %0, {%1, %2};" : "=l"(x) : "r"(w[q] << 16), "r"(w[q] & 0xffff0000u));
        asm("fma.rn.f32x2 %0, %1, %1, %0;" : "+l"(acc) : "l"(x));
    }
    asm("mov.b64 {%0, %1}, %2;" : "=f"(a0), "=f"(a1) : "l"(acc));
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
