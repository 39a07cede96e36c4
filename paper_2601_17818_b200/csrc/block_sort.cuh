// Block-wide bitonic sort of 64-bit keys, shared by the quota selection and the cluster-merge planner.
#pragma once

#include <stdint.h>

namespace vitcop {

// Bitonic sort of P = E * T 64-bit keys held E per thread by the first T threads of the CTA (T a multiple of
// 32, P a power of two), blocked: key p = t * E + e sits in slot e of thread t.  Compare-exchange partners at
// distance j < E are two slots of one thread; at distance j = m * E they are the same slot of threads t and
// t ^ m -- two lanes of a warp for m < 32 (shuffles), two warps otherwise (exchanged through `sm`, P keys).
// All threads of the CTA must call; on return sm[p] holds the ascending order.
template <int E, int J>
__device__ __forceinline__ void bitonic_local(unsigned long long (&r)[E], int base, int k) {
#pragma unroll
    for (int e = 0; e < E; ++e) {
        if ((e & J) == 0 && (e | J) < E) {
            const bool up = ((base + e) & k) == 0;
            const unsigned long long a = r[e], c = r[e | J];
            if ((a > c) == up) { r[e] = c; r[e | J] = a; }
        }
    }
}

// Barrier over the first `count` threads of the CTA (a multiple of 32), leaving the other warps out.
__device__ __forceinline__ void active_bar_sync(int count) { asm volatile("bar.sync 1, %0;" ::"r"(count) : "memory"); }

template <int E>
__device__ void block_bitonic_sort(unsigned long long (&r)[E], unsigned long long* sm, int T) {
    const int t = threadIdx.x;
    const int P = E * T;
    const int base = t * E;
    // Warps that hold no keys skip the network altogether: spinning through its empty iterations would take
    // issue slots away from the few warps that do the work when P is small.
    if (t < T) {
        for (int k = 2; k <= P; k <<= 1) {
            for (int j = k >> 1; j > 0; j >>= 1) {
                if (j < E) {
                    if (j == 1) bitonic_local<E, 1>(r, base, k);
                    else if (j == 2) bitonic_local<E, 2>(r, base, k);
                    else if (j == 4) bitonic_local<E, 4>(r, base, k);
                    else bitonic_local<E, 8>(r, base, k);
                    continue;
                }
                const int m = j / E;                       // partner thread is t ^ m
                const bool lower = (t & m) == 0;
                const bool up = (base & k) == 0;           // k > j >= E: the same for all slots of a thread
                const bool want_min = lower == up;
                if (m < 32) {
#pragma unroll
                    for (int e = 0; e < E; ++e) {
                        const unsigned long long o = __shfl_xor_sync(0xffffffffu, r[e], m);
                        r[e] = (want_min == (o < r[e])) ? o : r[e];
                    }
                } else {
#pragma unroll
                    for (int e = 0; e < E; ++e) sm[e * T + t] = r[e];
                    active_bar_sync(T);
#pragma unroll
                    for (int e = 0; e < E; ++e) {
                        const unsigned long long o = sm[e * T + (t ^ m)];
                        r[e] = (want_min == (o < r[e])) ? o : r[e];
                    }
                    active_bar_sync(T);
                }
            }
        }
#pragma unroll
        for (int e = 0; e < E; ++e) sm[base + e] = r[e];
    }
    __syncthreads();
}

}  // namespace vitcop
