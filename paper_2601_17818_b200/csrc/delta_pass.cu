// Eq. 3 (Algorithm 2, step 2) from stored Gram tiles: per token the nearest denser token inside the spatial radius.
//
// The density sweep (gram.cu, GRAM_RHO) has just computed every Gram value on the tensor cores and written the tiles
// it visited to the workspace; the densities it produces order the tokens, so Eq. 3 needs a second look at every
// pair.  Reading a pair back costs 4 bytes; recomputing it costs 2 D flop, several times more of the machine.  This
// kernel therefore streams the tiles from memory (L2 for the smaller problems, HBM for the long ones) and does the
// per-pair work of Eq. 3 with plain ALU instructions -- the same arithmetic, in the same order, as the delta epilogue
// of the one-kernel sweep, so both give the same bits.
//
// One CTA of 8 warps per tile, up to four CTAs per SM, a persistent grid; every CTA takes one contiguous run of the
// tile numbering, i.e. consecutive row blocks against one column block (see below why).  Warp w owns
// the rows 32 (w % 4) .. + 31 of the tile (one per lane) and the column half w / 4; a thread walks its half eight
// columns at a time (two 16-byte loads, the next four already in flight) and keeps its row's minimum; the minimum of
// a column is kept in shared memory.  The two halves of a row are combined through shared memory (ties keep the lower
// index) and rows and columns are folded into the per-token packed minima with one 64-bit atomicMin each.
//
// Most pairs cannot matter: a pair serves its row token only if its d^2 does not exceed the best that token has so
// far, and its column token likewise (and a pair serves only one of the two: the less dense one).  Both bounds are read from the packed minima when the tile starts (other CTAs
// keep lowering them, a stale bound is merely looser) and tightened as the tile goes.  A thread first computes d^2 of
// its eight pairs and tests them against the two bounds (with <=: an equal distance at a lower index still wins);
// one redux.or tells the warp whether any of its 256 pairs passed, and only the lanes whose pair passed go through
// the spatial test and update the row's minimum (in registers) or the column's (a packed 64-bit minimum in shared
// memory: smaller distance first, then the lower row).  What is skipped could not
// have changed any minimum, so the result is the same as without the test.
// The bounds only bite once a token has seen some of its candidates, so the order of the work matters: a CTA walks
// down one column block, whose tokens thus meet their candidates one row block after the other (their bounds stay in
// shared memory from tile to tile), while the CTAs of other column blocks reach any given row block at different
// times, so that a row token's bound in global memory has been lowered by the time most of them read it.
#include "gram.cuh"

namespace vitcop {
namespace {

constexpr int BM = kGramBM;
constexpr int kDpSlices = 2;                              // column slices of a tile, four warps each
constexpr int kDpThreads = 128 * kDpSlices;
constexpr int kDpCtasPerSm = 3;
constexpr float kInf = __builtin_huge_valf();

// Bits of the largest d^2 that can still improve the packed minimum at `p` (an equal d^2 with a lower index would):
// the d^2 it holds, or +inf when it holds none.  Read from L2: other CTAs lower it while this one runs.
__device__ __forceinline__ int bound_of(const unsigned long long* p) {
    const unsigned long long v = __ldcg(p);
    return v == ~0ull ? 0x7f800000 : (int)(uint32_t)(v >> 32);
}

__device__ __forceinline__ float4 ld_tile(const float4* p) {
    float4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                 : "l"(p));
    return v;
}

template <int BN, int METRIC, bool SPATIAL>
__global__ void __launch_bounds__(kDpThreads, kDpCtasPerSm)
delta_pass_kernel(const GramArgs g, const GramTiling tl, const long long total_tiles) {
    constexpr int NS = kDpSlices;
    constexpr int kSliceCols = BN / NS;
    constexpr int kGroups = kSliceCols / 8;
    __shared__ __align__(16) float colw[BN], cola[BN], colrho[BN], colx[BN], coly[BN];
    __shared__ __align__(16) int colthr[BN];               // bits of the largest d^2 that can still serve column j
    __shared__ unsigned long long colbest[BN];             // packed (d^2 bits, row) minimum of every column of the tile
    __shared__ float rowred[(kDpSlices - 1) * BM];
    __shared__ int rowidx[(kDpSlices - 1) * BM];
    __shared__ float roww[BM], rowa[BM], rowrho[BM], rowx[BM], rowy[BM];

    // A kernel queued behind this one that does not depend on it may share the SMs from the start.
    grid_dependency_launch_dependents();
    grid_dependency_wait();                                // rho, the factors and the tiles come from the preceding kernels

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int quarter = warp & 3, slice = warp >> 2;
    const int rl = quarter * 32 + lane;                    // tile-local row of this thread

    // Tiles whose row block lies beyond the spatial radius of their column blocks were not kept by the density sweep
    // and are not read here: g.kept lists the numbers of the others in ascending order (filter.cu), and the CTAs
    // share that list out evenly.  Without a radius every tile is kept and the list is the identity.
    const long long n_list = g.kept ? (long long)*g.n_kept : total_tiles;
    const long long k_begin = n_list * blockIdx.x / gridDim.x;
    const int run = (int)(n_list * (blockIdx.x + 1) / gridDim.x - k_begin);     // this CTA's entries: k_begin + [0, run)
    if (run <= 0) return;                                  // (uniform)
    const int32_t* const kept = g.kept ? g.kept + k_begin : nullptr;
    auto tile_of = [&](int k) { return kept ? (long long)kept[k] : k_begin + k; };
    __shared__ long long s_next;                           // number of the tile after the current one (-1: none)
    int k = 0;
    long long t = tile_of(0);
    // The thread's loads form one stream over the tiles of the run: the sixteen columns it works on (A, B: eight
    // each) and the sixteen after those, requested while it works -- across tile boundaries, so that the constants of
    // a new tile are fetched with data already in flight.  `pf` walks that stream: two float4 columns of 128 rows per
    // group; after a tile's last group it moves on to the next tile that is kept (s_next; null after the last).
    constexpr size_t kGroupStep = 2 * BM;                                      // float4 per group
    const float4* const tiles0 = reinterpret_cast<const float4*>(g.gram_tiles) + (size_t)(slice * kSliceCols / 4) * BM + rl;
    auto tile_ptr = [&](long long tt) { return tiles0 + (size_t)tt * (gram_tile_floats(BN) / 4); };
    const float4* pf = tile_ptr(t);
    float4 A0 = make_float4(0.f, 0.f, 0.f, 0.f), A1 = A0, B0 = A0, B1 = A0;
    int pf_group = 0;                                      // group inside its tile that pf points at
    auto fetch_pair = [&](float4& x0, float4& x1, float4& y0, float4& y1) {    // the next two groups of the stream
        if (pf) {
            x0 = ld_tile(pf);
            x1 = ld_tile(pf + BM);
            y0 = ld_tile(pf + kGroupStep);
            y1 = ld_tile(pf + kGroupStep + BM);
            pf += 2 * kGroupStep;
        }
        pf_group += 2;
        if (pf_group == kGroups) {
            pf_group = 0;
            const long long tn = s_next;
            pf = tn >= 0 ? tile_ptr(tn) : nullptr;
        }
    };
    fetch_pair(A0, A1, B0, B1);
    int prev_b = -1, prev_tj = -1;
    for (; k < run; ++k) {
        int b, ti, tj;
        decode_sym_tile(tl, t, b, ti, tj);
        if (threadIdx.x == 0) s_next = k + 1 < run ? tile_of(k + 1) : -1;   // (published by the barrier behind the tile's constants)
        const bool same_cols = b == prev_b && tj == prev_tj;       // the column block of the previous tile: its constants stay
        prev_b = b;
        prev_tj = tj;
        const int I0 = ti * BM, J0 = tj * BN;
        const int i = I0 + rl;
        const bool row_valid = i < g.n;
        const size_t bo = (size_t)b * g.n;

        for (int it = threadIdx.x; it < 2 * BN + 2 * BM; it += kDpThreads) {
            if (it < BN) {
                const int j = J0 + it;
                const bool cv = j < g.n;
                const int bound = cv ? bound_of(g.best + bo + j) : (int)0x80000000;
                colbest[it] = ~0ull;
                if (same_cols) {
                    colthr[it] = min(colthr[it], bound);
                } else {
                    colthr[it] = bound;
                    colw[it] = cv ? g.w[bo + j] : 0.f;
                    if (METRIC == 1) cola[it] = cv ? g.a[bo + j] : 0.f;
                }
            } else if (it < 2 * BN) {
                if (same_cols) continue;
                const int ce = it - BN, j = J0 + ce;
                float rj = 0.f;
                float2 pj = make_float2(0.f, 0.f);
                if (j < g.n) {
                    if (SPATIAL) pj = *reinterpret_cast<const float2*>(g.pos + 2 * (bo + j));
                    rj = g.rho[bo + j];
                }
                colrho[ce] = rj;
                if (SPATIAL) { colx[ce] = pj.x; coly[ce] = pj.y; }
            } else if (it < 2 * BN + BM) {
                const int r = it - 2 * BN, ir = I0 + r;
                const bool rv = ir < g.n;
                roww[r] = rv ? g.w[bo + ir] : 0.f;
                if (METRIC == 1) rowa[r] = rv ? g.a[bo + ir] : 0.f;
            } else {
                const int r = it - 2 * BN - BM, ir = I0 + r;
                float rr = 0.f;
                float2 pr = make_float2(0.f, 0.f);
                if (ir < g.n) {
                    if (SPATIAL) pr = *reinterpret_cast<const float2*>(g.pos + 2 * (bo + ir));
                    rr = g.rho[bo + ir];
                }
                rowrho[r] = rr;
                if (SPATIAL) { rowx[r] = pr.x; rowy[r] = pr.y; }
            }
        }
        // every pair of the tile has i < j < n: no masking needed
        const bool full = (J0 >= I0 + BM) && (J0 + BN <= g.n);
        __syncthreads();

        const float w_i = roww[rl];
        const float a_i = METRIC == 1 ? rowa[rl] : 1.f;
        const float m2w_i = -2.f * w_i;
        const float rho_i = rowrho[rl];
        float x_i = 0.f, y_i = 0.f;
        if (SPATIAL) { x_i = rowx[rl]; y_i = rowy[rl]; }

        float rbest = kInf;                                // row-side minimum and its tile-local column
        int rbest_c = -1;
        int rthr = row_valid ? bound_of(g.best + bo + i) : (int)0x80000000;   // bits of the largest d^2 that can still serve row i
        // One group: eight columns of this thread's row.
        auto group = [&](const float4& c0, const float4& c1, const int cl0) {
            const float v[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
            // ---- every pair: d^2 and the test against ONE bound, that of the less dense of the two tokens (the only
            //      one the pair can serve).  d^2 = a_i + a_j - 2 (g w_j) w_i, the operations and their order as in the
            //      one-kernel sweep.  Compared as signed integers, a (rounding-level) negative d^2, which the full
            //      treatment clamps to zero, passes every bound, as zero would.
            float d2v[8];
            uint32_t cand = 0;                             // bit u: column u of the group passed
#pragma unroll
            for (int q4 = 0; q4 < 2; ++q4) {
                const float4 cw = *reinterpret_cast<const float4*>(colw + cl0 + 4 * q4);
                const float4 cr = *reinterpret_cast<const float4*>(colrho + cl0 + 4 * q4);
                const int4 ct = *reinterpret_cast<const int4*>(colthr + cl0 + 4 * q4);
                float4 ca = make_float4(0.f, 0.f, 0.f, 0.f);
                if (METRIC == 1) ca = *reinterpret_cast<const float4*>(cola + cl0 + 4 * q4);
                const float cwv[4] = {cw.x, cw.y, cw.z, cw.w};
                const float crv[4] = {cr.x, cr.y, cr.z, cr.w};
                const float cav[4] = {ca.x, ca.y, ca.z, ca.w};
                const int ctv[4] = {ct.x, ct.y, ct.z, ct.w};
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    const int u = 4 * q4 + r;
                    const float x = v[u] * cwv[r];
                    d2v[u] = fmaf(x, m2w_i, METRIC == 0 ? 2.f : a_i + cav[r]);
                    if (__float_as_int(d2v[u]) <= (crv[r] > rho_i ? rthr : ctv[r])) cand |= 1u << u;
                }
            }
            // ---- the pairs that passed: spatial radius, then the row's own minimum (registers) or the column's (shared
            //      memory, packed so that the smaller distance and then the lower row wins).  Only the lanes that hold
            //      such a pair take the branch; one redux.or lets a warp without any skip the lot.
            const uint32_t live = __reduce_or_sync(0xffffffffu, cand);     // columns in which some lane's pair passed
            if (live == 0u) return;
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                if (!(live >> u & 1u)) continue;           // warp-uniform: a column nobody needs costs one branch
                if (!(cand >> u & 1u)) continue;
                const int ce = cl0 + u;
                bool usable = true;                        // the pair may serve as (child, parent) at all
                if (SPATIAL) {
                    const float dx = colx[ce] - x_i, dy = coly[ce] - y_i;
                    usable = fmaf(dx, dx, dy * dy) <= g.tau2;
                }
                if (!full) {
                    const int j = J0 + ce;
                    usable = usable && j > i && j < g.n && row_valid;
                }
                if (!usable) continue;
                const float d2 = fmaxf(d2v[u], 0.f);
                // with i < j: "j denser than i" is rho_j > rho_i, "i denser than j" is its complement
                if (colrho[ce] > rho_i) {                  // j as parent candidate of i (row side)
                    if (d2 < rbest) {                      // (columns come in ascending order: ties keep the lower one)
                        rbest = d2;
                        rbest_c = ce;
                        rthr = __float_as_int(d2);
                    }
                } else {                                   // i as parent candidate of j (column side)
                    atomicMin(colbest + ce, ((unsigned long long)__float_as_uint(d2) << 32) | (unsigned long long)(uint32_t)i);
                    atomicMin(colthr + ce, __float_as_int(d2));
                }
            }
        };
#pragma unroll 2
        for (int c = 0; c < kGroups; c += 2) {
            float4 N0 = A0, N1 = A1, M0 = B0, M1 = B1;
            fetch_pair(N0, N1, M0, M1);
            group(A0, A1, slice * kSliceCols + c * 8);
            group(B0, B1, slice * kSliceCols + c * 8 + 8);
            A0 = N0; A1 = N1; B0 = M0; B1 = M1;
        }

        const long long t_next = s_next;                   // (rewritten only behind the barriers below)
        // ---- combine the four column slices of every row and the four row quarters of every column
        if (slice > 0) {
            rowred[(slice - 1) * BM + rl] = rbest;
            rowidx[(slice - 1) * BM + rl] = rbest_c;
        }
        __syncthreads();
        if (slice == 0 && row_valid) {
#pragma unroll
            for (int q = 0; q < NS - 1; ++q) {             // ascending columns: ties keep the lower one
                const float other = rowred[q * BM + rl];
                if (other < rbest) { rbest = other; rbest_c = rowidx[q * BM + rl]; }
            }
            if (rbest_c >= 0)
                atomicMin(g.best + bo + i, ((unsigned long long)__float_as_uint(rbest) << 32) |
                                               (unsigned long long)(uint32_t)(J0 + rbest_c));
        }
        for (int ce = threadIdx.x; ce < BN; ce += kDpThreads) {
            const unsigned long long cb = colbest[ce];
            if (cb != ~0ull && J0 + ce < g.n) atomicMin(g.best + bo + J0 + ce, cb);
        }
        __syncthreads();                                   // the shared arrays are rewritten for the next tile
        t = t_next;
    }
}

template <int BN, int METRIC, bool SPATIAL>
int launch_dp(const GramArgs& g, const GramTiling& tl, long long total, cudaStream_t stream, bool pdl, int ctas_per_sm) {
    cudaLaunchConfig_t cfg = {};
    const long long ctas = (long long)ctas_per_sm * gram_num_sms();
    cfg.gridDim = dim3((unsigned)(total < ctas ? total : ctas));
    cfg.blockDim = dim3(kDpThreads);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_allowed(pdl) ? 1 : 0;
    KernelTimeScope timed("delta_pass_kernel", stream);
    return record_cuda(cudaLaunchKernelEx(&cfg, delta_pass_kernel<BN, METRIC, SPATIAL>, g, tl, total));
}

template <int BN>
int launch_dp_bn(const GramArgs& g, const GramTiling& tl, long long total, cudaStream_t stream, bool pdl, int cps) {
    const bool euclid = g.metric == 1;
    const bool spatial = g.tau2 >= 0.f && g.pos != nullptr;
    if (spatial)
        return euclid ? launch_dp<BN, 1, true>(g, tl, total, stream, pdl, cps)
                      : launch_dp<BN, 0, true>(g, tl, total, stream, pdl, cps);
    return euclid ? launch_dp<BN, 1, false>(g, tl, total, stream, pdl, cps)
                  : launch_dp<BN, 0, false>(g, tl, total, stream, pdl, cps);
}

}  // namespace

int launch_delta_pass(const GramArgs& args, const GramTiling& tiling, cudaStream_t stream, bool pdl, bool leave_room) {
    const long long total = (long long)args.B * tiling.tiles_per_b;
    if (total <= 0) return VITCOP_OK;
    if (!args.gram_tiles || !args.best) return VITCOP_ERR_INVALID_ARG;
    // (`leave_room`: a kernel that runs beside this one finds a third of every SM's registers and thread slots free)
    const int cps = kDpCtasPerSm; (void)leave_room;
    if (tiling.BN != 256) return VITCOP_ERR_INVALID_ARG;   // (long samples always take the wide tiles)
    return launch_dp_bn<256>(args, tiling, total, stream, pdl, cps);
}

}  // namespace vitcop
