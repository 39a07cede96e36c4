// Redundancy filter = Visual Information Clustering (Algorithm 2, Eq. 2 and Eq. 3) on one B200.
//
// Pipeline (one stream, no host synchronisation; consecutive kernels overlap through programmatic dependent
// launch, each waiting for its predecessor before it reads what that one wrote):
//   1. Gram sweep, GRAM_DIAG  the diagonal tiles only: g_ii -> per-token factors (cosine: 1/sqrt(g_ii);
//                             euclid: g_ii), from the same tensor-core arithmetic as every g_ij
//   2. Gram sweep, GRAM_RHO   Gram tiles on the tensor cores (gram.cu); the epilogue turns each tile into
//                             squared distances, exp(-(d/d_c)^2) and partial sums of Eq. 2 per tile, and, for
//                             long samples, keeps the tile's Gram values in the workspace
//   3. rho_reduce_kernel      fixed-order sum of the partials -> rho (bit-reproducible)
//   4. delta_pass_kernel      (long samples) reads the tiles back (delta_pass.cu) and keeps, per token, the nearest
//                             denser token inside the spatial radius (Eq. 3) as a packed (d^2, j) 64-bit minimum;
//      Gram sweep, GRAM_DELTA (otherwise) the same tiles computed again, Eq. 3 in the epilogue
//   5. vic_finalize_kernel    gamma = rho * delta, radix-select of the centres, pointer jumping over the
//                             parent forest, orphan fallback, labels (Algorithm 2, steps 3-4)
// Small problems replace 1-4 by gram_resident_kernel (gram.cu): one pass over the Gram tiles, accumulators kept in
// tensor memory.
#include "gram.cuh"

namespace vitcop {
namespace {

// ------------------------------------------------------------------------------------------------
// small kernels
// ------------------------------------------------------------------------------------------------
// rho[b,i] = sum of the partials of the tiles that hold token i, in a fixed order (reproducible bits): the row-side
// slots of the column tiles that pair row tile i / 128 with later tokens, then the column-side slots of the row tiles
// that pair column tile i / BN with earlier tokens -- one contiguous range of slots.  LANES neighbouring lanes share a
// token: each adds its part of the range slot by slot (sixteen independent loads at a time), and the sums are added
// in lane order.  A long sample has up to 190 slots per token, which one thread alone would fetch in a dozen
// dependent rounds; for a few dozen slots one thread per token is the faster shape.
constexpr int kRhoLanesLong = 4;
constexpr int kRhoLongSlots = 64;                          // samples with more slots than this take kRhoLanesLong lanes
template <int LANES>
__global__ void rho_reduce_kernel(const float* __restrict__ part, int n, GramTiling t, float* __restrict__ rho,
                                  float* __restrict__ rho_user) {
    grid_dependency_launch_dependents();
    grid_dependency_wait();
    const int q = threadIdx.x % LANES;
    const int i = (blockIdx.x * blockDim.x + threadIdx.x) / LANES;
    const int b = blockIdx.y;
    const bool valid = i < n;                              // (all lanes stay for the shuffles)
    float s = 0.f;
    if (valid) {
        const int ti = i / kGramBM, tj = i / t.BN;
        const int cap = t.R * (tj + 1);
        const int first = ti / t.R, last = t.TJ + (t.TI < cap ? t.TI : cap);
        const int per = (last - first + LANES - 1) / LANES;
        const int c0 = first + q * per, c1 = min(last, c0 + per);
        const float* p = part + (size_t)b * t.slots() * t.n_pad + i;
        for (int c = c0; c < c1; c += 16) {
            float v[16];
#pragma unroll
            for (int u = 0; u < 16; ++u) v[u] = (c + u < c1) ? p[(size_t)(c + u) * t.n_pad] : 0.f;
#pragma unroll
            for (int u = 0; u < 16; ++u)
                if (c + u < c1) s += v[u];
        }
    }
    float others[LANES];
#pragma unroll
    for (int u = 1; u < LANES; ++u) others[u] = __shfl_down_sync(0xffffffffu, s, u);
    if (!valid || q != 0) return;
#pragma unroll
    for (int u = 1; u < LANES; ++u) s += others[u];
    rho[(size_t)b * n + i] = s;
    if (rho_user) rho_user[(size_t)b * n + i] = s;
}

// The tiles of the symmetric numbering that lie within the spatial radius (gram.cuh: tile_outside_radius), in
// ascending order: list[0 .. *count).  One small CTA that fits on an SM beside a CTA of the density sweep: it is
// queued behind that sweep, does its work while the sweep runs and only then waits for it, so that the kernels
// queued behind see both complete.  Thread t tests the tiles [t E, (t + 1) E) of a round of 256 E tiles with all its
// loads in flight; one scan per round places them.
constexpr int kKeptThreads = 256;
constexpr int kKeptPerThread = 16;
__global__ void __launch_bounds__(kKeptThreads)
kept_tiles_kernel(const float4* __restrict__ bbox, GramTiling t, long long total, float tau2, int32_t* __restrict__ list,
                  int32_t* __restrict__ count) {
    __shared__ uint32_t warp_sums[kKeptThreads / 32];
    grid_dependency_launch_dependents();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t placed = 0;
    for (long long base = 0; base < total; base += (long long)kKeptThreads * kKeptPerThread) {
        uint32_t keep = 0;
#pragma unroll
        for (int e = 0; e < kKeptPerThread; ++e) {
            const long long tile = base + (long long)threadIdx.x * kKeptPerThread + e;
            if (tile < total) {
                int b, ti, tj;
                decode_sym_tile(t, tile, b, ti, tj);
                if (!tile_outside_radius(bbox + (size_t)b * t.TI, t, ti, tj, tau2)) keep |= 1u << e;
            }
        }
        // exclusive prefix of the per-thread counts over the CTA, in thread order
        const uint32_t mine = __popc(keep);
        uint32_t incl = mine;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const uint32_t o = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off) incl += o;
        }
        __syncthreads();                                   // (the previous round's sums have been read)
        if (lane == 31) warp_sums[warp] = incl;
        __syncthreads();
        uint32_t before = 0, round_total = 0;
#pragma unroll
        for (int w = 0; w < kKeptThreads / 32; ++w) {
            const uint32_t v = warp_sums[w];
            if (w < warp) before += v;
            round_total += v;
        }
        uint32_t pos = placed + before + incl - mine;
#pragma unroll
        for (int e = 0; e < kKeptPerThread; ++e)
            if (keep >> e & 1u) list[pos++] = (int32_t)(base + (long long)threadIdx.x * kKeptPerThread + e);
        placed += round_total;
    }
    if (threadIdx.x == 0) *count = (int32_t)placed;
    grid_dependency_wait();
}

// ------------------------------------------------------------------------------------------------
// Centres, forest roots and labels: one CTA per sample.
// ------------------------------------------------------------------------------------------------
constexpr int kFinThreads = 1024;
constexpr int kFinIters = VITCOP_MAX_VISUAL_TOKENS / kFinThreads;      // tokens per thread at the largest sample

// Shared memory: keys[n] (uint64; later reused as next[n] int32), isc[n] (uint8), centres[nc] (int32).
__global__ void __launch_bounds__(kFinThreads)
vic_finalize_kernel(const uint16_t* __restrict__ feat, int n, int D, int n_centers, const float* __restrict__ rho,
                    const unsigned long long* __restrict__ best, const float* __restrict__ w,
                    const float* __restrict__ a, int32_t* __restrict__ label, int32_t* __restrict__ n_clusters,
                    float* __restrict__ delta2_user, int32_t* __restrict__ parent_user) {
    extern __shared__ __align__(16) uint8_t fin_smem[];
    unsigned long long* keys = reinterpret_cast<unsigned long long*>(fin_smem);
    int32_t* nxt = reinterpret_cast<int32_t*>(fin_smem);              // aliases keys after the selection
    uint8_t* isc = fin_smem + (size_t)n * 8;
    int32_t* centres = reinterpret_cast<int32_t*>(fin_smem + (size_t)n * 8 + (((size_t)n + 15) & ~(size_t)15));
    __shared__ uint32_t hist[256];
    __shared__ uint32_t warp_sums[32];
    __shared__ uint32_t cnt[kFinIters * 32];               // one count per (iteration, warp)
    __shared__ uint32_t s_digit, s_krem, s_whole;
    __shared__ unsigned long long orph_best[kFinThreads];
    __shared__ int orph_list[kFinThreads];
    __shared__ int orph_cnt;

    grid_dependency_launch_dependents();
    grid_dependency_wait();
    const int b = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    rho += (size_t)b * n;
    best += (size_t)b * n;
    w += (size_t)b * n;
    a += (size_t)b * n;
    label += (size_t)b * n;
    feat += (size_t)b * n * D;
    if (delta2_user) delta2_user += (size_t)b * n;
    if (parent_user) parent_user += (size_t)b * n;
    const int nc = min(n_centers, n);

    // rank key, ascending = better centre candidate: ~( orphan ? (0xFFFFFFFF, rho) : (gamma, rho) )
    for (int i = tid; i < n; i += kFinThreads) {
        const unsigned long long p = best[i];
        const bool orphan = p == ~0ull;
        const float d2 = orphan ? __int_as_float(0x7f800000) : __uint_as_float((uint32_t)(p >> 32));
        const int par = orphan ? -1 : (int)(uint32_t)(p & 0xFFFFFFFFull);
        if (delta2_user) delta2_user[i] = d2;
        if (parent_user) parent_user[i] = par;
        const float r = rho[i];
        const uint32_t hi = orphan ? 0xFFFFFFFFu : __float_as_uint(r * sqrtf(d2));
        keys[i] = ~(((unsigned long long)hi << 32) | (unsigned long long)__float_as_uint(r));
    }
    __syncthreads();

    // ---- radix select of the nc smallest keys (8 passes of 8 bits), ties -> lower index
    unsigned long long T = ~0ull;
    uint32_t krem = 0;
    if (nc > 0 && nc < n) {
        unsigned long long prefix = 0;
        krem = (uint32_t)nc;
        for (int pass = 0; pass < 8; ++pass) {
            const int shift = 56 - 8 * pass;
            const unsigned long long hi_mask = pass == 0 ? 0ull : (~0ull << (shift + 8));
            if (tid < 256) hist[tid] = 0;
            __syncthreads();
            for (int base = 0; base < n; base += kFinThreads) {
                const int i = base + tid;
                int dig = -1;
                if (i < n) {
                    const unsigned long long key = keys[i];
                    if ((key & hi_mask) == prefix) dig = (int)((key >> shift) & 255ull);
                }
                const uint32_t peers = __match_any_sync(0xffffffffu, dig);
                if (dig >= 0 && lane == __ffs(peers) - 1) atomicAdd(&hist[dig], (uint32_t)__popc(peers));
            }
            __syncthreads();
            const uint32_t c = tid < 256 ? hist[tid] : 0u;
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
                for (int q = 0; q < warp; ++q) basew += warp_sums[q];
                const uint32_t incl = basew + v, excl = incl - c;
                if (excl < krem && krem <= incl) {
                    s_digit = (uint32_t)tid;
                    s_krem = krem - excl;
                    s_whole = (c == krem - excl) ? 1u : 0u;         // the whole bin is wanted
                }
            }
            __syncthreads();
            prefix |= (unsigned long long)s_digit << shift;
            krem = s_krem;
            const bool whole = s_whole != 0;
            __syncthreads();
            if (whole) {
                // every key that shares the prefix found so far is selected: no need to resolve lower digits
                prefix |= (1ull << shift) - 1ull;
                krem = 0xFFFFFFFFu;
                break;
            }
        }
        T = prefix;
    }
    // ---- centre flags + ascending centre list.  Token i = it * 1024 + tid; ranks in index order come from one count
    //      per (iteration, warp), scanned once for the whole sample, plus the lane's position in its warp's ballot:
    //      first among the keys equal to the cut (ties -> lower index), then among the centres.
    {
        uint32_t eq_mask = 0, f_mask = 0;                  // bit it: this thread's token of iteration it is ... / is a centre
        const int iters = (n + kFinThreads - 1) / kFinThreads;          // <= kFinIters
        const uint32_t lane_below = (1u << lane) - 1u;
        const bool cut = nc > 0 && nc < n;
        if (cut) {
            for (int it = 0; it < iters; ++it) {
                const int i = it * kFinThreads + tid;
                const bool eq = i < n && keys[i] == T;
                const uint32_t bal = __ballot_sync(0xffffffffu, eq);
                if (eq) eq_mask |= 1u << it;
                if (lane == 0) cnt[it * 32 + warp] = __popc(bal);
            }
            __syncthreads();
            uint32_t total;
            const uint32_t excl = block_exclusive_sum(tid < iters * 32 ? cnt[tid] : 0u, warp_sums, total);
            if (tid < iters * 32) cnt[tid] = excl;
            __syncthreads();
        }
        for (int it = 0; it < iters; ++it) {
            const int i = it * kFinThreads + tid;
            bool f;
            if (nc <= 0) f = false;
            else if (nc >= n) f = i < n;
            else {
                const bool eq = (eq_mask >> it & 1u) != 0;
                const uint32_t bal = __ballot_sync(0xffffffffu, eq);
                const uint32_t eq_rank = cnt[it * 32 + warp] + __popc(bal & lane_below);
                f = i < n && (keys[i] < T || (eq && eq_rank < krem));
            }
            if (f) f_mask |= 1u << it;
            if (i < n) isc[i] = f ? 1 : 0;
        }
        __syncthreads();                                   // cnt is reused
        for (int it = 0; it < iters; ++it) {
            const uint32_t bal = __ballot_sync(0xffffffffu, (f_mask >> it & 1u) != 0);
            if (lane == 0) cnt[it * 32 + warp] = __popc(bal);
        }
        __syncthreads();
        uint32_t total;
        const uint32_t excl = block_exclusive_sum(tid < iters * 32 ? cnt[tid] : 0u, warp_sums, total);
        if (tid < iters * 32) cnt[tid] = excl;
        __syncthreads();
        for (int it = 0; it < iters; ++it) {
            const bool f = (f_mask >> it & 1u) != 0;
            const uint32_t bal = __ballot_sync(0xffffffffu, f);
            const uint32_t r = cnt[it * 32 + warp] + __popc(bal & lane_below);
            if (f && r < (uint32_t)nc) centres[r] = it * kFinThreads + tid;
        }
    }
    __syncthreads();   // keys are dead from here on; nxt aliases them

    // ---- forest roots by pointer jumping: a centre or an orphan is its own root
    for (int i = tid; i < n; i += kFinThreads) {
        const unsigned long long p = best[i];
        const int par = (p == ~0ull) ? -1 : (int)(uint32_t)(p & 0xFFFFFFFFull);
        nxt[i] = (isc[i] || par < 0 || par >= n) ? i : par;
    }
    __syncthreads();
    for (int round = 0; round < 16; ++round) {
        int changed = 0;
        for (int i = tid; i < n; i += kFinThreads) {
            const int p = nxt[i];
            const int q = nxt[p];
            if (q != p) {
                nxt[i] = q;       // any value read here is an ancestor of i, roots are fixed points
                changed = 1;
            }
        }
        if (!__syncthreads_or(changed)) break;
    }

    // ---- labels; a root that is an orphan but not a centre joins the nearest centre (feature distance)
    for (int i = tid; i < n; i += kFinThreads) {
        const int root = nxt[i];
        label[i] = isc[root] ? root : -1 - root;
    }
    __syncthreads();
    int any_surplus = 0;                                   // a root that is neither a centre nor below one
    for (int i = tid; i < n; i += kFinThreads) any_surplus |= (!isc[i] && nxt[i] == i) ? 1 : 0;
    any_surplus = __syncthreads_or(any_surplus);
    if (nc > 0 && any_surplus) {
        // Surplus orphans (roots that are not centres) are rare but each needs its distance to every centre: they
        // are listed, kFinThreads tokens at a time, and the (orphan, centre) pairs are spread over all warps; the
        // nearest centre wins through a packed minimum (distance bits, then the lower centre rank).
        for (int base = 0; base < n; base += kFinThreads) {
            __syncthreads();                                        // the previous round's list has been consumed
            if (tid == 0) orph_cnt = 0;
            __syncthreads();
            const int o = base + tid;
            if (o < n && !isc[o] && nxt[o] == o) {
                const int at = atomicAdd(&orph_cnt, 1);
                orph_list[at] = o;
                orph_best[at] = ~0ull;
            }
            __syncthreads();
            const int pairs = orph_cnt * nc;
            for (int pr = warp; pr < pairs; pr += kFinThreads / 32) {
                const int e = pr / nc, q = pr - e * nc;
                const int oo = orph_list[e], c = centres[q];
                const uint16_t* fo = feat + (size_t)oo * D;
                const uint16_t* fc = feat + (size_t)c * D;
                float dot = 0.f;
                for (int k = lane * 2; k < D; k += 64) {
                    const uint32_t u = *reinterpret_cast<const uint32_t*>(fo + k);
                    const uint32_t v = *reinterpret_cast<const uint32_t*>(fc + k);
                    dot = fmaf(bf16lo(u), bf16lo(v), dot);
                    dot = fmaf(bf16hi(u), bf16hi(v), dot);
                }
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
                const float d2 = fmaxf(0.f, fmaf(-2.f, (dot * w[oo]) * w[c], a[oo] + a[c]));
                if (lane == 0)
                    atomicMin(&orph_best[e], ((unsigned long long)__float_as_uint(d2) << 32) | (unsigned long long)q);
            }
            __syncthreads();
            if (tid < orph_cnt)                                     // remember the adopted centre at the root
                nxt[orph_list[tid]] = -1 - centres[(int)(orph_best[tid] & 0xFFFFFFFFull)];
        }
    }
    __syncthreads();
    for (int i = tid; i < n; i += kFinThreads) {
        const int l = label[i];
        if (l < 0) {
            const int root = -1 - l;
            const int adopted = nxt[root];
            label[i] = adopted < 0 ? -1 - adopted : root;
        }
    }
    if (tid == 0) n_clusters[b] = nc;
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
// Workspace of the filter: status block | row-block flags [B, ceil(n / 128)] | w | a | rho | best |
// rho partials [B, slots, n_pad] (sized for either tile width) | bounding boxes of the row blocks' positions |
// count and list of the tiles within the spatial radius | Gram tiles of the density sweep (problems too large
// for the one-kernel sweep: 4 bytes per pair of the symmetric half, tile padding included).  The status block and the
// flags are zeroed at the start of every call.  Words of the status block: 0 status, 2 grid barrier.
struct FilterWs {
    size_t off_flags, off_w, off_a, off_rho, off_best, off_part, off_bbox, off_kept, off_tiles, total;
    FilterWs(int B, int n) {
        size_t o = kStatusBytes;
        const size_t bn = (size_t)B * n;
        off_flags = o; o += align_up((size_t)B * ((n + kGramBM - 1) / kGramBM) * 4, 256);
        off_w = o;    o += align_up(bn * 4, 256);
        off_a = o;    o += align_up(bn * 4, 256);
        off_rho = o;  o += align_up(bn * 4, 256);
        off_best = o; o += align_up(bn * 8, 256);
        const GramTiling t = make_gram_tiling(n, 128);           // the narrow tiling has the most slots
        off_part = o; o += align_up((size_t)B * t.slots() * t.n_pad * 4, 256);
        off_bbox = o;   o += align_up((size_t)B * t.TI * sizeof(float4), 256);
        off_kept = off_tiles = o;
        if (gram_keeps_tiles(B, n)) {
            const int bn = gram_pick_bn(B, n);
            const size_t tiles = (size_t)B * make_gram_tiling(n, bn).tiles_per_b;
            o += align_up((tiles + 1) * sizeof(int32_t), 256);    // count, then the list of kept tiles
            off_tiles = o;
            o += align_up(tiles * gram_tile_floats(bn) * 4, 256);
        }
        total = o;
    }
};

void pdl_config(cudaLaunchConfig_t& cfg, cudaLaunchAttribute* attr, dim3 grid, dim3 block, size_t smem,
                cudaStream_t stream, bool pdl) {
    cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_allowed(pdl) ? 1 : 0;
}

}  // namespace

size_t filter_zeroed_bytes(int B, int n) { return FilterWs(B, n).off_w; }

size_t filter_workspace_bytes(int B, int n, int D) {
    (void)D;
    return FilterWs(B, n).total;
}
size_t similarity_workspace_bytes(int B, int n, int D) {
    (void)D;
    return kStatusBytes + 2 * align_up((size_t)B * n * 4, 256);
}

int launch_filter(const void* feat, const float* pos, int B, int n, int D, const vitcop_filter_params& p,
                  int n_centers, int32_t* label, int32_t* n_clusters, float* rho_user, float* delta2_user,
                  int32_t* parent_user, void* workspace, cudaStream_t stream, const KnormJob* knorm) {
    FilterWs l(B, n);
    char* ws = static_cast<char*>(workspace);
    float* w = reinterpret_cast<float*>(ws + l.off_w);
    float* a = reinterpret_cast<float*>(ws + l.off_a);
    float* rho = reinterpret_cast<float*>(ws + l.off_rho);
    unsigned long long* best = reinterpret_cast<unsigned long long*>(ws + l.off_best);
    float* part = reinterpret_cast<float*>(ws + l.off_part);

    const GramTiling tiling = make_gram_tiling(n, gram_pick_bn(B, n));
    GramArgs g = {};
    g.B = B; g.n = n; g.D = D; g.row0 = 0; g.row_end = n; g.metric = p.metric;
    g.c2 = -1.4426950408889634f / (p.d_c * p.d_c);
    g.tau2 = (p.tau >= 0.f && pos) ? p.tau * p.tau : -1.f;
    g.w = w; g.a = a; g.rho = rho; g.pos = pos; g.part = part; g.best = best;
    g.w_out = w; g.a_out = a;
    g.sim_out = nullptr; g.status = reinterpret_cast<int*>(ws);

    // The first kernel of the call is launched without programmatic overlap, so everything queued before the call
    // (the producer of the features included) has completed when it starts.
    int rc;
    int knorm_in_sweep = 0;                                // leading samples whose K-norm the Gram sweep computes
    const bool resident = gram_fits_resident(B, n);
    if (resident) {
        g.rho_out = rho;
        g.rho_user = rho_user;
        g.grid_sync = reinterpret_cast<unsigned int*>(ws) + 2;       // zeroed with the status word at the start of the call
        g.diag_ready = reinterpret_cast<unsigned int*>(ws + l.off_flags);
        if (knorm && gram_resident_takes_knorm(knorm->H, knorm->d)) {
            // The sweep's two idle warps take the K-norm of the first samples, about as many as they finish while
            // the epilogue warps work on the accumulators; the other samples follow beside vic_finalize_kernel.
            knorm_in_sweep = (5 * knorm->B + 8) / 16;
            if (knorm_in_sweep > 0) {
                g.kn_K = knorm->K; g.kn_score = knorm->score; g.kn_B = knorm_in_sweep;
                g.kn_H = knorm->H; g.kn_N = knorm->N; g.kn_d = knorm->d; g.kn_vis_start = knorm->vis_start; g.kn_Nv = knorm->Nv;
            }
        }
        rc = launch_gram_resident(feat, g, make_gram_tiling(n, 128), stream);
        if (rc != VITCOP_OK) return rc;
    } else {
        const bool keep_tiles = gram_keeps_tiles(B, n);
        g.gram_tiles = keep_tiles ? reinterpret_cast<float*>(ws + l.off_tiles) : nullptr;
        // with a spatial radius, tiles beyond it are neither kept nor read back (gram.cuh: tile_outside_radius)
        g.bbox = (keep_tiles && g.tau2 >= 0.f) ? reinterpret_cast<float4*>(ws + l.off_bbox) : nullptr;
        rc = launch_gram_sweep(GRAM_DIAG, feat, g, make_gram_tiling(n, 128), stream, false);
        if (rc != VITCOP_OK) return rc;
        rc = launch_gram_sweep(GRAM_RHO, feat, g, tiling, stream, true);
        if (rc != VITCOP_OK) return rc;
        if (g.bbox) {
            // which tiles the delta pass will read: one small CTA beside the density sweep (the boxes come from the
            // diagonal sweep, complete since the density sweep's epilogues started)
            int32_t* cnt = reinterpret_cast<int32_t*>(ws + l.off_kept);
            const long long tiles = (long long)B * tiling.tiles_per_b;
            if (tiles > 0x7fffffffLL) return VITCOP_ERR_UNSUPPORTED;
            cudaLaunchConfig_t cfg;
            cudaLaunchAttribute attr[1];
            pdl_config(cfg, attr, dim3(1), dim3(kKeptThreads), 0, stream, true);
            KernelTimeScope timed("kept_tiles_kernel", stream);
            rc = record_cuda(cudaLaunchKernelEx(&cfg, kept_tiles_kernel, (const float4*)g.bbox, tiling, tiles, g.tau2, cnt + 1,
                                                cnt));
            if (rc != VITCOP_OK) return rc;
            g.kept = cnt + 1;
            g.n_kept = cnt;
        }
        {
            cudaLaunchConfig_t cfg;
            cudaLaunchAttribute attr[1];
            const int lanes = tiling.slots() > kRhoLongSlots ? kRhoLanesLong : 1;
            pdl_config(cfg, attr, dim3((n * lanes + 255) / 256, B), dim3(256), 0, stream, true);
            KernelTimeScope timed("rho_reduce_kernel", stream);
            rc = record_cuda(cudaLaunchKernelEx(&cfg, lanes == 1 ? rho_reduce_kernel<1> : rho_reduce_kernel<kRhoLanesLong>,
                                                (const float*)part, n, tiling, rho, rho_user));
            if (rc != VITCOP_OK) return rc;
        }
        if (!keep_tiles) {
            rc = launch_gram_sweep(GRAM_DELTA, feat, g, tiling, stream, true);
            if (rc != VITCOP_OK) return rc;
        }
        // The delta pass is bound by ALU issue and by the read of the tiles, the K-norm by the read of K: given one,
        // the pass leaves a quarter of every SM free and the K-norm, which depends on nothing in this call, runs
        // beside it (it still waits for the pass before it ends, so the kernels behind it see both complete).
        const bool knorm_beside = keep_tiles && knorm != nullptr;
        if (keep_tiles) {
            rc = launch_delta_pass(g, tiling, stream, true, knorm_beside);
            if (rc != VITCOP_OK) return rc;
        }
        if (knorm_beside) {
            rc = launch_knorm(knorm->K, knorm->B, knorm->H, knorm->d, (int64_t)knorm->H * knorm->N * knorm->d,
                              (int64_t)knorm->N * knorm->d, knorm->d, knorm->vis_start, nullptr, knorm->Nv, knorm->score,
                              knorm->Nv, stream, true);
            if (rc != VITCOP_OK) return rc;
            knorm_in_sweep = knorm->B;                     // nothing left for the launch behind vic_finalize_kernel
        }
    }

    const int nc = n_centers < n ? n_centers : n;
    const size_t smem = (size_t)n * 8 + (((size_t)n + 15) & ~(size_t)15) + (size_t)(nc > 0 ? nc : 1) * 4 + 16;
    if (smem > 32 * 1024) {                                // (the kernel's static arrays take part of the default 48 KB)
        cudaError_t e = cudaFuncSetAttribute(vic_finalize_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return record_cuda(e);
    }
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    pdl_config(cfg, attr, dim3(B), dim3(kFinThreads), smem, stream, true);
    {
        KernelTimeScope timed("vic_finalize_kernel", stream);
        rc = record_cuda(cudaLaunchKernelEx(&cfg, vic_finalize_kernel, static_cast<const uint16_t*>(feat), n, D, nc,
                                            (const float*)rho, (const unsigned long long*)best, (const float*)w,
                                            (const float*)a, label, n_clusters, delta2_user, parent_user));
        if (rc != VITCOP_OK) return rc;
    }
    if (knorm && knorm_in_sweep < knorm->B) {
        // vic_finalize_kernel runs one CTA per sample and releases its dependents when it starts: the K-norm, which
        // does not depend on the clustering, streams K from HBM on the other SMs meanwhile and waits for the
        // finalize kernel before it ends.  (Beside the Gram sweep it would not fit: that kernel's CTAs hold most
        // of each SM's registers.)
        const int64_t stride_b = (int64_t)knorm->H * knorm->N * knorm->d;
        rc = launch_knorm(static_cast<const uint16_t*>(knorm->K) + (size_t)knorm_in_sweep * stride_b,
                          knorm->B - knorm_in_sweep, knorm->H, knorm->d, stride_b, (int64_t)knorm->N * knorm->d, knorm->d,
                          knorm->vis_start, nullptr, knorm->Nv, knorm->score + (size_t)knorm_in_sweep * knorm->Nv,
                          knorm->Nv, stream, true);
    }
    return rc;
}

int launch_similarity_rows(const void* feat, int B, int n, int D, int metric, int row_begin, int row_end, float* out,
                           void* workspace, cudaStream_t stream) {
    char* ws = static_cast<char*>(workspace);
    float* w = reinterpret_cast<float*>(ws + kStatusBytes);
    float* a = reinterpret_cast<float*>(ws + kStatusBytes + align_up((size_t)B * n * 4, 256));
    GramArgs g = {};
    g.B = B; g.n = n; g.D = D; g.row0 = row_begin; g.row_end = row_end; g.metric = metric;
    g.c2 = 0.f; g.tau2 = -1.f;
    g.w = w; g.a = a; g.w_out = w; g.a_out = a; g.sim_out = out; g.status = reinterpret_cast<int*>(ws);
    int rc = launch_gram_sweep(GRAM_DIAG, feat, g, make_gram_tiling(n, 128), stream, false);
    if (rc != VITCOP_OK) return rc;
    return launch_gram_sweep(GRAM_SIM, feat, g, make_gram_tiling(n, 128), stream, true);
}

}  // namespace vitcop
