// CPU oracle for the ViTCoP visual-token pruning operator chain (arXiv 2601.17818).
//
// TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, fp64 statement of what the
// paper defines, written from its equations and pseudocode.  It shares no code, header,
// table or helper with the CUDA library and must never be called from the product path;
// only the tests, the smoke check and the benchmark's CPU-baseline leg may load it.
//
// Conventions
//   * bf16 tensors arrive as uint16 bit patterns; widening to double is exact.
//   * every sum, norm, similarity and distance is computed in double.
//   * "OpenMP" appears only as `parallel for` over independent output rows / samples;
//     no sum is split, blocked or reordered by it.
//   * all functions are per call stateless; outputs are caller-allocated.
//
// Readings of the paper adopted where it is silent:
//   R1  density order is total: j is "denser" than i iff rho_j > rho_i, or rho_j == rho_i and j < i
//       (Eq. 3 / Algorithm 2 step 2 print a strict ">" which leaves exact duplicates unordered).
//   R2  a token with no admissible denser neighbour ("orphan", delta = +inf, N_i = -1) ranks first
//       when centres are chosen (gamma = rho * inf); orphans among themselves by rho desc, index asc.
//   R3  non-centres inherit the label of N_i in descending density order (Algorithm 2 step 4);
//       an orphan that is not a centre takes the nearest centre by feature distance
//       (the main text's assignment rule, Section "VIC Algorithm").
//   R4  a label is the token index of its cluster's centre (Algorithm 2 numbers them 1..N_centers;
//       the partition is the same).
//   R5  top-k ties go to the lower index; kept tokens are reported in ascending index order.
//   R6  the quota of Eq. 5 is evaluated in exact integer arithmetic: q_c = (|C_c| * (B - N_c)) div n.
//   R7  NaN scores sort after every number (they are pruned first when the smallest are kept).
//   R8  merged rows (Eq. 6) come out in ascending order of their cluster label; where they are placed in the
//       sequence is left to the caller (Algorithm 3 returns an unordered union).
//   R9  the softmax of Eq. 1 runs over all keys of the layer, the [CLS] key included; scores are reported for
//       the visual tokens only.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <numeric>
#include <vector>

namespace {

inline double bf16_to_double(uint16_t b) {
    uint32_t u = static_cast<uint32_t>(b) << 16;
    float f;
    std::memcpy(&f, &u, sizeof f);
    return static_cast<double>(f);
}

// (score, index) order used by every top-k in the paper: ascending score, NaN last, ties -> lower index.
inline bool score_less(double a, int ia, double b, int ib) {
    const bool na = std::isnan(a), nb = std::isnan(b);
    if (na != nb) return nb;            // a number precedes NaN
    if (!na && a != b) return a < b;
    return ia < ib;
}

// R1: is token j denser than token i ?
inline bool denser(const double* rho, int j, int i) {
    return rho[j] > rho[i] || (rho[j] == rho[i] && j < i);
}

}  // namespace

extern "C" {

// ---------------------------------------------------------------------------------------------
// O1. K-norm saliency, Eq. 4:  ||K_i||_2 = sqrt( sum_h ||K_i^(h)||_2^2 )  for the visual tokens.
//   K      bf16 bits, element (b,h,t,e) at b*stride_b + h*stride_h + t*stride_n + e
//   score  [B, Nv_cap] doubles; entries past a sample's vis_len are left untouched
// ---------------------------------------------------------------------------------------------
void oracle_knorm(const uint16_t* K, int B, int H, int N, int d, int64_t stride_b, int64_t stride_h,
                  int64_t stride_n, int vis_start, const int32_t* vis_len, int vis_len_uniform,
                  double* score, int Nv_cap) {
    (void)N;
#pragma omp parallel for schedule(static)
    for (int b = 0; b < B; ++b) {
        const int nv = vis_len ? vis_len[b] : vis_len_uniform;
        for (int i = 0; i < nv; ++i) {
            double acc = 0.0;
            for (int h = 0; h < H; ++h) {
                const uint16_t* row = K + b * stride_b + h * stride_h + (int64_t)(vis_start + i) * stride_n;
                for (int e = 0; e < d; ++e) {
                    const double v = bf16_to_double(row[e]);
                    acc += v * v;
                }
            }
            score[(int64_t)b * Nv_cap + i] = std::sqrt(acc);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// O2. Plain top-k (Algorithm 1, Stage III: TopK(V, -K_norms, k); Stage I uses largest = 1).
//   Keeps k' = min(budget, n) tokens: the first k' in (score asc, index asc) order -- or
//   (score desc, index asc) when largest != 0 -- and writes them in ascending index order.
//   Returns k'.
// ---------------------------------------------------------------------------------------------
int oracle_select_plain(const double* score, int n, int budget, int largest, int32_t* keep_idx) {
    std::vector<int> order(n);
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
        const double sa = largest ? -score[a] : score[a];
        const double sb = largest ? -score[b] : score[b];
        return score_less(sa, a, sb, b);
    });
    const int k = std::max(0, std::min(budget, n));
    std::vector<int> kept(order.begin(), order.begin() + k);
    std::sort(kept.begin(), kept.end());
    for (int r = 0; r < k; ++r) keep_idx[r] = kept[r];
    return k;
}

// ---------------------------------------------------------------------------------------------
// O4. Cluster-quota selection (Eq. 5, Algorithm 3 up to the elite set; merging is not done here).
//   N_c = number of distinct labels; B_elites = budget - N_c; q_c = (|C_c| * B_elites) div n;
//   inside each cluster the q_c smallest scores are kept (ties -> lower index).
//   Writes the union in ascending index order; returns its size, or -1 when budget < N_c.
//   n_clusters_out (optional) receives N_c;  quota_out (optional, [n]) receives q_c at the
//   position of each cluster's label value (0 elsewhere).
// ---------------------------------------------------------------------------------------------
int oracle_select_quota(const double* score, const int32_t* label, int n, int budget, int32_t* keep_idx,
                        int32_t* n_clusters_out, int32_t* quota_out) {
    std::vector<int32_t> labs(label, label + n);
    std::sort(labs.begin(), labs.end());
    labs.erase(std::unique(labs.begin(), labs.end()), labs.end());
    const int Nc = static_cast<int>(labs.size());
    if (n_clusters_out) *n_clusters_out = Nc;
    if (quota_out) std::fill(quota_out, quota_out + n, 0);
    if (budget < Nc) return -1;
    const int64_t B_elites = budget - Nc;
    std::vector<int> kept;
    for (int c = 0; c < Nc; ++c) {
        std::vector<int> members;
        for (int i = 0; i < n; ++i)
            if (label[i] == labs[c]) members.push_back(i);
        const int64_t size_c = static_cast<int64_t>(members.size());
        int64_t q = (size_c * B_elites) / n;
        if (q > size_c) q = size_c;
        if (quota_out && labs[c] >= 0 && labs[c] < n) quota_out[labs[c]] = static_cast<int32_t>(q);
        std::stable_sort(members.begin(), members.end(),
                         [&](int a, int b) { return score_less(score[a], a, score[b], b); });
        for (int64_t r = 0; r < q; ++r) kept.push_back(members[r]);
    }
    std::sort(kept.begin(), kept.end());
    for (size_t r = 0; r < kept.size(); ++r) keep_idx[r] = kept[r];
    return static_cast<int>(kept.size());
}

// ---------------------------------------------------------------------------------------------
// O3a. Pairwise feature "distance" (Algorithm 2, step 1, first line) for one sample.
//   gram   g_ij = sum_e f_ie f_je
//   metric 0 (cosine): s_ij = g_ij / sqrt(g_ii g_jj); d2_ij = max(0, 2 - 2 s_ij)   (squared distance
//            between the L2-normalised features); a zero-norm feature has s = 0 against everything.
//   metric 1 (euclid): d2_ij = max(0, g_ii + g_jj - 2 g_ij).
//   Writes rows [row_begin, row_end) of the n x n matrices d2 and/or sim (either may be NULL);
//   sim is s_ij for metric 0 and the raw g_ij for metric 1.  Row r of the output is token row_begin + r.
// ---------------------------------------------------------------------------------------------
void oracle_feature_distance_rows(const uint16_t* feat, int n, int D, int metric, int row_begin, int row_end,
                                  double* d2, double* sim) {
    std::vector<float> f(static_cast<size_t>(n) * D);       // exact widening, keeps the inner loop readable
    for (size_t t = 0; t < f.size(); ++t) f[t] = static_cast<float>(bf16_to_double(feat[t]));
    std::vector<double> gdiag(n);
    for (int i = 0; i < n; ++i) {
        double acc = 0.0;
        const float* a = &f[static_cast<size_t>(i) * D];
        for (int e = 0; e < D; ++e) acc += static_cast<double>(a[e]) * static_cast<double>(a[e]);
        gdiag[i] = acc;
    }
#pragma omp parallel for schedule(dynamic, 4)
    for (int i = row_begin; i < row_end; ++i) {
        const float* a = &f[static_cast<size_t>(i) * D];
        const size_t o = static_cast<size_t>(i - row_begin) * n;
        for (int j = 0; j < n; ++j) {
            const float* c = &f[static_cast<size_t>(j) * D];
            double g = 0.0;
            for (int e = 0; e < D; ++e) g += static_cast<double>(a[e]) * static_cast<double>(c[e]);
            double s, dist2;
            if (metric == 0) {
                const double den = std::sqrt(gdiag[i] * gdiag[j]);
                s = den > 0.0 ? g / den : 0.0;
                dist2 = std::max(0.0, 2.0 - 2.0 * s);
            } else {
                s = g;
                dist2 = std::max(0.0, gdiag[i] + gdiag[j] - 2.0 * g);
            }
            if (d2) d2[o + j] = dist2;
            if (sim) sim[o + j] = s;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// O3b. Local density, Eq. 2:  rho_i = sum_{j != i} exp( -(d_ij / d_c)^2 ).   d2 is n x n.
// ---------------------------------------------------------------------------------------------
void oracle_vic_density(const double* d2, int n, double d_c, double* rho) {
#pragma omp parallel for schedule(static)
    for (int i = 0; i < n; ++i) {
        double acc = 0.0;
        for (int j = 0; j < n; ++j) {
            if (j == i) continue;
            acc += std::exp(-d2[static_cast<size_t>(i) * n + j] / (d_c * d_c));
        }
        rho[i] = acc;
    }
}

// ---------------------------------------------------------------------------------------------
// O3c. delta and nearest denser neighbour, Eq. 3 / Algorithm 2 step 2.
//   Over j denser than i (R1) with ||p_i - p_j||_2 <= tau:  delta_i = min d_ij, N_i = argmin
//   (ties -> lowest j).  pos == NULL or tau < 0 disables the spatial test.  No admissible j:
//   delta2_i = +inf, parent_i = -1.
//   Optional robustness report for comparing against a lower-precision implementation:
//   fragile[i] = 1 when a perturbation of rho by a relative tol_rho, of d2 by tol_d2_abs +
//   tol_d2_rel * d2, or of the spatial distance by a relative tol_sp could change parent_i.
// ---------------------------------------------------------------------------------------------
void oracle_vic_parents(const double* d2, const float* pos, const double* rho, int n, double tau,
                        double* delta2, int32_t* parent, uint8_t* fragile, double tol_rho, double tol_d2_abs,
                        double tol_d2_rel, double tol_sp) {
    const bool spatial = pos != nullptr && tau >= 0.0;
    const double inf = std::numeric_limits<double>::infinity();
#pragma omp parallel for schedule(static)
    for (int i = 0; i < n; ++i) {
        double best = inf;
        int bj = -1;
        for (int j = 0; j < n; ++j) {
            if (j == i || !denser(rho, j, i)) continue;
            if (spatial) {
                const double dx = static_cast<double>(pos[2 * i]) - static_cast<double>(pos[2 * j]);
                const double dy = static_cast<double>(pos[2 * i + 1]) - static_cast<double>(pos[2 * j + 1]);
                if (std::sqrt(dx * dx + dy * dy) > tau) continue;
            }
            const double v = d2[static_cast<size_t>(i) * n + j];
            if (v < best) { best = v; bj = j; }
        }
        delta2[i] = best;
        parent[i] = bj;
        if (!fragile) continue;
        // Could a small perturbation change the answer?
        bool frag = false;
        const double band = (bj >= 0) ? best + tol_d2_abs + tol_d2_rel * best : inf;
        for (int j = 0; j < n && !frag; ++j) {
            if (j == i) continue;
            const double m = tol_rho * std::max(std::fabs(rho[i]), std::fabs(rho[j]));
            const bool maybe_denser = rho[j] >= rho[i] - m;
            const bool surely_denser = rho[j] > rho[i] + m;
            bool maybe_near = true, surely_near = true;
            if (spatial) {
                const double dx = static_cast<double>(pos[2 * i]) - static_cast<double>(pos[2 * j]);
                const double dy = static_cast<double>(pos[2 * i + 1]) - static_cast<double>(pos[2 * j + 1]);
                const double sp = std::sqrt(dx * dx + dy * dy);
                maybe_near = sp <= tau * (1.0 + tol_sp);
                surely_near = sp <= tau * (1.0 - tol_sp);
            }
            if (j == bj) {
                if (!(surely_denser && surely_near)) frag = true;
            } else if (maybe_denser && maybe_near) {
                if (d2[static_cast<size_t>(i) * n + j] <= band) frag = true;
            }
        }
        fragile[i] = frag ? 1 : 0;
    }
}

// ---------------------------------------------------------------------------------------------
// O3d. Cluster centres, Algorithm 2 step 3:  gamma = rho * delta; the n_centers tokens with the
//   largest gamma are centres.  Rank key (R2): orphans first (gamma = +inf), then gamma desc,
//   then rho desc, then index asc.  gamma_out (optional) receives rho_i * sqrt(delta2_i).
//   rank_out (optional, [n]) receives the token indices in rank order.
// ---------------------------------------------------------------------------------------------
void oracle_vic_centers(const double* rho, const double* delta2, int n, int n_centers, uint8_t* is_center,
                        double* gamma_out, int32_t* rank_out) {
    const double inf = std::numeric_limits<double>::infinity();
    std::vector<double> gamma(n);
    for (int i = 0; i < n; ++i) gamma[i] = std::isinf(delta2[i]) ? inf : rho[i] * std::sqrt(delta2[i]);
    std::vector<int> order(n);
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
        if (gamma[a] != gamma[b]) return gamma[a] > gamma[b];
        if (rho[a] != rho[b]) return rho[a] > rho[b];
        return a < b;
    });
    const int nc = std::max(0, std::min(n_centers, n));
    std::fill(is_center, is_center + n, 0);
    for (int r = 0; r < nc; ++r) is_center[order[r]] = 1;
    if (gamma_out) std::copy(gamma.begin(), gamma.end(), gamma_out);
    if (rank_out) std::copy(order.begin(), order.end(), rank_out);
}

// ceil(n * alpha) of Algorithm 2 step 3, evaluated in double; clamped to [0, n].
int oracle_vic_num_centers(int n, double alpha) {
    const double v = std::ceil(static_cast<double>(n) * alpha);
    return static_cast<int>(std::max(0.0, std::min(static_cast<double>(n), v)));
}

// ---------------------------------------------------------------------------------------------
// O3e. Label assignment, Algorithm 2 step 4 (R3, R4).  Centres label themselves; the others are
//   visited in descending density order and copy the label of their parent; an orphan that is
//   not a centre copies the nearest centre by d2 (ties -> lowest centre index).
//   Needs n_centers >= 1 whenever n >= 1 (otherwise labels stay -1).
// ---------------------------------------------------------------------------------------------
void oracle_vic_labels(const double* d2, const double* rho, const int32_t* parent, const uint8_t* is_center,
                       int n, int32_t* label) {
    std::vector<int> order(n);
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return denser(rho, a, b); });
    for (int i = 0; i < n; ++i) label[i] = is_center[i] ? i : -1;
    for (int t = 0; t < n; ++t) {
        const int i = order[t];
        if (label[i] != -1) continue;
        if (parent[i] >= 0) {
            label[i] = label[parent[i]];
        } else {
            double best = std::numeric_limits<double>::infinity();
            int bc = -1;
            for (int c = 0; c < n; ++c) {
                if (!is_center[c]) continue;
                const double v = d2[static_cast<size_t>(i) * n + c];
                if (v < best) { best = v; bc = c; }
            }
            label[i] = bc;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// O5. Order-preserving compaction of one sample: output rows are the input rows at positions
//   [0, vis_start), then vis_start + keep_idx[r] (r ascending), then [vis_start + vis_len, seq_len).
//   hidden [N, Dh], K and V [H, N, d] (row strides N*d per head), outputs with Ncap rows.
//   Rows are copied as bytes.  Returns out_len = seq_len - vis_len + n_keep.
// ---------------------------------------------------------------------------------------------
int oracle_compact(const uint16_t* hidden, const uint16_t* K, const uint16_t* V, int H, int N, int d, int Dh,
                   int seq_len, int vis_start, int vis_len, const int32_t* keep_idx, int n_keep,
                   uint16_t* hidden_out, uint16_t* K_out, uint16_t* V_out, int Ncap, int32_t* kept_pos) {
    std::vector<int> src;
    for (int t = 0; t < vis_start; ++t) src.push_back(t);
    for (int r = 0; r < n_keep; ++r) src.push_back(vis_start + keep_idx[r]);
    for (int t = vis_start + vis_len; t < seq_len; ++t) src.push_back(t);
    const int out_len = static_cast<int>(src.size());
    for (int r = 0; r < out_len; ++r) {
        const int t = src[r];
        if (kept_pos) kept_pos[r] = t;
        if (hidden && hidden_out)
            std::memcpy(hidden_out + static_cast<size_t>(r) * Dh, hidden + static_cast<size_t>(t) * Dh,
                        sizeof(uint16_t) * Dh);
        for (int h = 0; h < H; ++h) {
            if (K && K_out)
                std::memcpy(K_out + (static_cast<size_t>(h) * Ncap + r) * d, K + (static_cast<size_t>(h) * N + t) * d,
                            sizeof(uint16_t) * d);
            if (V && V_out)
                std::memcpy(V_out + (static_cast<size_t>(h) * Ncap + r) * d, V + (static_cast<size_t>(h) * N + t) * d,
                            sizeof(uint16_t) * d);
        }
    }
    return out_len;
}

// Budget arithmetic of Algorithm 1: floor(m * pi), evaluated in double.
int oracle_stage_count(int m, double pi) { return static_cast<int>(std::floor(static_cast<double>(m) * pi)); }

// Integrated token compression ratio, Eq. 10.
double oracle_cr_int(double pi1, double pi2, double pi3, int l_s, int l_d, int n_layers) {
    const double kept = pi1 * (l_s - 1) + pi2 * (l_d - l_s) + pi3 * (n_layers - l_d + 1);
    return 1.0 - kept / n_layers;
}

// ---------------------------------------------------------------------------------------------
// O7. Cluster merge, Eq. 6 / Algorithm 3 second half, for one sample: every cluster's tokens that were NOT
//   kept as elites are averaged into one representative row,
//       t_c^merged = (1 / |C_c^remaining|) * sum_{i in C_c^remaining} t_i .
//   hidden [N, Dh] bf16 bits, the visual span starts at vis_start and has n tokens; label[n], keep[n] (1 = elite).
//   Clusters are visited in ascending label value; a cluster without remaining tokens yields no row.
//   merged [Mcap, Dh] doubles, merged_label / merged_count [Mcap]; returns the number of merged rows.
//   (Where the merged rows go in the sequence is the caller's choice: Algorithm 3 returns a set.)
// ---------------------------------------------------------------------------------------------
int oracle_merge_clusters(const uint16_t* hidden, int N, int Dh, int vis_start, int n, const int32_t* label,
                          const uint8_t* keep, double* merged, int32_t* merged_label, int32_t* merged_count,
                          int Mcap) {
    (void)N;
    std::vector<int32_t> labs(label, label + n);
    std::sort(labs.begin(), labs.end());
    labs.erase(std::unique(labs.begin(), labs.end()), labs.end());
    int m = 0;
    for (int32_t lab : labs) {
        std::vector<int> rest;
        for (int i = 0; i < n; ++i)
            if (label[i] == lab && !keep[i]) rest.push_back(i);
        if (rest.empty()) continue;
        if (m < Mcap) {
            for (int e = 0; e < Dh; ++e) {
                double acc = 0.0;
                for (int i : rest) acc += bf16_to_double(hidden[static_cast<size_t>(vis_start + i) * Dh + e]);
                merged[static_cast<size_t>(m) * Dh + e] = acc / static_cast<double>(rest.size());
            }
            merged_label[m] = lab;
            merged_count[m] = static_cast<int32_t>(rest.size());
        }
        ++m;
    }
    return m;
}

// ---------------------------------------------------------------------------------------------
// O8. Stage I saliency, Eq. 1, for one image:  S_i = sum_h A^(h)_{0,i}, where A^(h) is the attention matrix
//   of head h of the vision encoder layer and row 0 belongs to the [CLS] token:
//       A^(h)_{0,j} = softmax_j( scale * q^(h) . k_j^(h) ),   j = 0 .. M-1   (key 0 is [CLS] itself).
//   q [H, d] is the [CLS] query, K [H, M, d] the keys (bf16 bits).  S [M-1] receives the scores of the visual
//   tokens j = 1 .. M-1; cls_out (optional) the attention [CLS] pays to itself, summed over heads.
// ---------------------------------------------------------------------------------------------
void oracle_cls_saliency(const uint16_t* q, const uint16_t* K, int H, int M, int d, double scale, double* S,
                         double* cls_out) {
    std::vector<double> total(M, 0.0), logit(M);
    for (int h = 0; h < H; ++h) {
        double mx = -std::numeric_limits<double>::infinity();
        for (int j = 0; j < M; ++j) {
            double acc = 0.0;
            for (int e = 0; e < d; ++e)
                acc += bf16_to_double(q[static_cast<size_t>(h) * d + e]) *
                       bf16_to_double(K[(static_cast<size_t>(h) * M + j) * d + e]);
            logit[j] = scale * acc;
            mx = std::max(mx, logit[j]);
        }
        double den = 0.0;
        for (int j = 0; j < M; ++j) den += std::exp(logit[j] - mx);
        for (int j = 0; j < M; ++j) total[j] += std::exp(logit[j] - mx) / den;
    }
    for (int j = 1; j < M; ++j) S[j - 1] = total[j];
    if (cls_out) *cls_out = total[0];
}

// ---------------------------------------------------------------------------------------------
// O9. The K vectors of Eq. 4 at their source: K^(h)_i = W_k^(h) t_i for every head (one row of W per output
//   feature, as a linear layer stores it), optionally rotated by rotary position embedding (pairs (e, e + d/2) of a
//   head turned by the angle whose cosine / sine the tables give at the token's position), and the K-norm of Eq. 4
//   taken on the bf16 values a K cache would hold.  One sample.
//   hidden [N, Dh] and W [H * d, Dh] are bf16 bit patterns; cos_tab / sin_tab [n_pos, d / 2] doubles or NULL (no
//   rotation); position [N] (NULL: token index).  Outputs: K64 [H, N, d] doubles (before rounding), K_bf16 [H, N, d]
//   bit patterns (round to nearest even), score [N] = sqrt(sum over heads and elements of the rounded values squared).
// ---------------------------------------------------------------------------------------------
static uint16_t double_to_bf16_rne(double v) {
    float f = static_cast<float>(v);                        // fp64 -> fp32 -> bf16: the double rounding can differ from a
    uint32_t u;                                             // direct one only on exact ties of the second step, which the
    std::memcpy(&u, &f, sizeof u);                          // first step's 29 discarded bits make vanishingly rare
    if ((u & 0x7fffffffu) > 0x7f800000u) return static_cast<uint16_t>((u >> 16) | 0x40);   // NaN stays NaN
    const uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return static_cast<uint16_t>(u >> 16);
}

void oracle_kproj_knorm(const uint16_t* hidden, const uint16_t* W, int N, int Dh, int H, int d, const double* cos_tab,
                        const double* sin_tab, const int32_t* position, double* K64, uint16_t* K_bf16, double* score) {
    const int half = d / 2;
#pragma omp parallel for schedule(static)
    for (int t = 0; t < N; ++t) {
        std::vector<double> row(static_cast<size_t>(H) * d);
        for (int c = 0; c < H * d; ++c) {
            double acc = 0.0;
            for (int k = 0; k < Dh; ++k)
                acc += bf16_to_double(hidden[static_cast<size_t>(t) * Dh + k]) * bf16_to_double(W[static_cast<size_t>(c) * Dh + k]);
            row[c] = acc;
        }
        if (cos_tab && sin_tab) {
            const int p = position ? position[t] : t;
            for (int h = 0; h < H; ++h)
                for (int e = 0; e < half; ++e) {
                    const double a = row[h * d + e], b = row[h * d + e + half];
                    const double c = cos_tab[static_cast<size_t>(p) * half + e], s = sin_tab[static_cast<size_t>(p) * half + e];
                    row[h * d + e] = a * c - b * s;
                    row[h * d + e + half] = b * c + a * s;
                }
        }
        double acc = 0.0;
        for (int h = 0; h < H; ++h)
            for (int e = 0; e < d; ++e) {
                const double v = row[h * d + e];
                const size_t o = (static_cast<size_t>(h) * N + t) * d + e;
                const uint16_t r = double_to_bf16_rne(v);
                if (K64) K64[o] = v;
                if (K_bf16) K_bf16[o] = r;
                const double q = bf16_to_double(r);
                acc += q * q;
            }
        score[t] = std::sqrt(acc);
    }
}

// Cost model of Appendix E.  Eq. 7: FLOPs of one transformer layer on a sequence of N tokens, hidden size d.
double oracle_flops_layer(double N, double d) { return 4.0 * N * N * d + 16.0 * N * d * d; }

// Eq. 8: visual tokens present at layer l (1-based) of an n-layer LLM: pi1*m before l_s, pi2*m from l_s, pi3*m from l_d.
double oracle_visual_tokens_at_layer(int l, double m, double pi1, double pi2, double pi3, int l_s, int l_d) {
    if (l < l_s) return pi1 * m;
    if (l < l_d) return pi2 * m;
    return pi3 * m;
}

// Eq. 9: total FLOPs of the LLM with the three-stage schedule (N_t text tokens ride along at every layer).
double oracle_flops_vitcop(double m, double n_text, double d, double pi1, double pi2, double pi3, int l_s, int l_d,
                           int n_layers) {
    return (l_s - 1) * oracle_flops_layer(pi1 * m + n_text, d) + (l_d - l_s) * oracle_flops_layer(pi2 * m + n_text, d) +
           (n_layers - l_d + 1) * oracle_flops_layer(pi3 * m + n_text, d);
}

}  // extern "C"
