// Public C ABI of libvitcop: argument validation, workspace carving and dispatch to the launchers.
#include <atomic>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <mutex>
#include <vector>

#include "gram.cuh"
#include "internal.cuh"

namespace vitcop {

static thread_local int g_last_cuda_error = 0;

int record_cuda(cudaError_t e) {
    if (e == cudaSuccess) return VITCOP_OK;
    g_last_cuda_error = static_cast<int>(e);
    return VITCOP_ERR_CUDA;
}

// ---- diagnostic kernel timing ------------------------------------------------------------------------
namespace {
struct TimedLaunch {
    const char* name;
    cudaEvent_t start, stop;
    bool complete;
};
std::atomic<bool> g_timing_on{false};
std::mutex g_timing_mutex;
std::vector<TimedLaunch> g_timed;
}  // namespace

bool kernel_timing_on() { return g_timing_on.load(std::memory_order_relaxed); }

KernelTimeScope::KernelTimeScope(const char* name, cudaStream_t stream) : slot_(-1), stream_(stream) {
    if (!kernel_timing_on()) return;
    TimedLaunch t{name, nullptr, nullptr, false};
    if (cudaEventCreate(&t.start) != cudaSuccess) return;
    if (cudaEventCreate(&t.stop) != cudaSuccess) { cudaEventDestroy(t.start); return; }
    cudaEventRecord(t.start, stream);
    std::lock_guard<std::mutex> lock(g_timing_mutex);
    slot_ = (int)g_timed.size();
    g_timed.push_back(t);
}

KernelTimeScope::~KernelTimeScope() {
    if (slot_ < 0) return;
    std::lock_guard<std::mutex> lock(g_timing_mutex);
    if (slot_ < (int)g_timed.size()) {
        cudaEventRecord(g_timed[slot_].stop, stream_);
        g_timed[slot_].complete = true;
    }
}

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool aligned8(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 7u) == 0; }
inline bool aligned256(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 255u) == 0; }

inline bool overlaps(const void* a, size_t na, const void* b, size_t nb) {
    if (!a || !b || na == 0 || nb == 0) return false;
    const uintptr_t x = reinterpret_cast<uintptr_t>(a), y = reinterpret_cast<uintptr_t>(b);
    return x < y + nb && y < x + na;
}

// Workspace of the fused step: status | score [B,Nv] | keep_idx [B,Nv] | n_keep [B]
struct StepWs {
    size_t off_score, off_keep, off_nkeep, total;
    StepWs(int B, int Nv) {
        size_t o = kStatusBytes;
        off_score = o; o += align_up((size_t)B * Nv * sizeof(float), 256);
        off_keep = o;  o += align_up((size_t)B * Nv * sizeof(int32_t), 256);
        off_nkeep = o; o += align_up((size_t)B * sizeof(int32_t), 256);
        total = o;
    }
};

int reset_status(void* ws, cudaStream_t s) { return record_cuda(cudaMemsetAsync(ws, 0, kStatusBytes, s)); }

int check_span(int N, int vis_start, const int32_t* vis_len, int vis_len_uniform, int Nv_cap) {
    if (vis_start < 0 || vis_start > N) return VITCOP_ERR_INVALID_ARG;
    if (!vis_len) {
        if (vis_len_uniform < 0 || vis_start + (int64_t)vis_len_uniform > N) return VITCOP_ERR_INVALID_ARG;
        if (Nv_cap >= 0 && vis_len_uniform > Nv_cap) return VITCOP_ERR_INVALID_ARG;
    } else if (Nv_cap >= 0 && vis_start + (int64_t)Nv_cap > N) {
        // device-side lengths are clamped to the capacity, which itself must fit the sequence
        return VITCOP_ERR_INVALID_ARG;
    }
    return VITCOP_OK;
}

}  // namespace
}  // namespace vitcop

using namespace vitcop;

// ---- built-in scratch of vitcop_prune_step_static ------------------------------------------------------
// Lives in every GPU that loads the library, from load to exit.  In host code the array's name is only a
// stand-in for the symbol, not a device address: the address each device gives it is looked up once per
// device with cudaGetSymbolAddress and that pointer is what the kernels receive.
constexpr size_t kStaticScratchBytes = VITCOP_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
void* g_scratch_addr[kMaxDevices] = {};

// Device address of g_static_scratch on the current device (looked up on the first call per device).
int static_scratch_address(void** out) {
    int dev = -1;
    int rc = record_cuda(cudaGetDevice(&dev));
    if (rc != VITCOP_OK) return rc;
    if (dev < 0 || dev >= kMaxDevices) return VITCOP_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        rc = record_cuda(cudaGetSymbolAddress(&p, g_static_scratch));
        if (rc != VITCOP_OK) return rc;
        if (!p) return VITCOP_ERR_CUDA;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return VITCOP_OK;
}
}  // namespace

extern "C" {

const char* vitcop_status_string(int status) {
    switch (status) {
        case VITCOP_OK: return "ok";
        case VITCOP_ERR_INVALID_ARG: return "invalid argument";
        case VITCOP_ERR_UNSUPPORTED: return "unsupported shape or alignment";
        case VITCOP_ERR_WORKSPACE: return "workspace missing or too small";
        case VITCOP_ERR_BUDGET: return "budget smaller than the number of clusters";
        case VITCOP_ERR_CUDA: return "CUDA runtime error";
        case VITCOP_ERR_TIMEOUT: return "bounded device wait expired";
        default: return "unknown status";
    }
}

int vitcop_last_cuda_error(void) { return g_last_cuda_error; }

int vitcop_set_wait_limit(unsigned long long limit_ns, int expire_roles) {
    gram_set_wait_debug(limit_ns, expire_roles);
    return VITCOP_OK;
}

int vitcop_kernel_timing_begin(void) {
    std::lock_guard<std::mutex> lock(g_timing_mutex);
    for (auto& t : g_timed) { cudaEventDestroy(t.start); cudaEventDestroy(t.stop); }
    g_timed.clear();
    g_timing_on.store(true);
    return VITCOP_OK;
}

int vitcop_kernel_timing_end(vitcop_kernel_time* out, int capacity, int* count) {
    if (!count || capacity < 0 || (capacity > 0 && !out)) return VITCOP_ERR_INVALID_ARG;
    g_timing_on.store(false);
    std::lock_guard<std::mutex> lock(g_timing_mutex);
    int n = 0, rc = VITCOP_OK;
    for (auto& t : g_timed) {
        float ms = 0.f;
        if (t.complete && rc == VITCOP_OK) {
            rc = record_cuda(cudaEventSynchronize(t.stop));
            if (rc == VITCOP_OK) rc = record_cuda(cudaEventElapsedTime(&ms, t.start, t.stop));
            if (rc == VITCOP_OK) {
                int k = 0;
                while (k < n && std::strncmp(out[k].name, t.name, sizeof(out[k].name) - 1) != 0) ++k;
                if (k == n && n < capacity) {
                    std::memset(&out[n], 0, sizeof(out[n]));
                    std::strncpy(out[n].name, t.name, sizeof(out[n].name) - 1);
                    ++n;
                }
                if (k < n) { out[k].launches += 1; out[k].total_ms += ms; }
            }
        }
        cudaEventDestroy(t.start);
        cudaEventDestroy(t.stop);
    }
    g_timed.clear();
    *count = n;
    return rc;
}

int vitcop_workspace_bytes(int op, int B, int H, int N, int d, int Nv, int D, int Dh, size_t* bytes) {
    (void)Dh;
    if (!bytes || B < 0 || Nv < 0 || D < 0) return VITCOP_ERR_INVALID_ARG;
    switch (op) {
        case VITCOP_OP_FILTER: *bytes = filter_workspace_bytes(B, Nv, D); return VITCOP_OK;
        case VITCOP_OP_SIMILARITY: *bytes = similarity_workspace_bytes(B, Nv, D); return VITCOP_OK;
        case VITCOP_OP_KNORM: *bytes = 0; return VITCOP_OK;
        case VITCOP_OP_COMPACT: *bytes = 0; return VITCOP_OK;
        case VITCOP_OP_SELECT: *bytes = kStatusBytes; return VITCOP_OK;
        case VITCOP_OP_PRUNE_STEP: *bytes = StepWs(B, Nv).total; return VITCOP_OK;
        case VITCOP_OP_COLLAB_STEP:
            *bytes = align_up(filter_workspace_bytes(B, Nv, D), 256) + StepWs(B, Nv).total;
            return VITCOP_OK;
        case VITCOP_OP_MERGE:
            if (N < 0) return VITCOP_ERR_INVALID_ARG;
            *bytes = merge_workspace_bytes(B, Nv, N);
            return VITCOP_OK;
        case VITCOP_OP_KPROJ:
            if (H < 0 || N < 0 || d < 0) return VITCOP_ERR_INVALID_ARG;
            *bytes = kproj_workspace_bytes(B, N, H, d);
            return VITCOP_OK;
        case VITCOP_OP_SALIENCY:
            if (H < 0 || N < 0) return VITCOP_ERR_INVALID_ARG;
            *bytes = saliency_workspace_bytes(B, H, N);
            return VITCOP_OK;
        default: return VITCOP_ERR_INVALID_ARG;
    }
}

int vitcop_poll_status(const void* workspace, void* stream, int* device_status) {
    if (!workspace || !device_status) return VITCOP_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int v = 0;
    int rc = record_cuda(cudaMemcpyAsync(&v, workspace, sizeof(int), cudaMemcpyDeviceToHost, s));
    if (rc != VITCOP_OK) return rc;
    rc = record_cuda(cudaStreamSynchronize(s));
    if (rc != VITCOP_OK) return rc;
    *device_status = v;
    return VITCOP_OK;
}

int vitcop_knorm_score(const void* K, int B, int H, int N, int d, int64_t stride_b, int64_t stride_h,
                       int64_t stride_n, int vis_start, const int32_t* vis_len, int vis_len_uniform, float* score,
                       int Nv_cap, void* stream) {
    if (!K || !score || B < 0 || H < 0 || N < 0 || d < 0 || Nv_cap < 0) return VITCOP_ERR_INVALID_ARG;
    if (stride_b < 0 || stride_h < 0 || stride_n < 0) return VITCOP_ERR_INVALID_ARG;
    int rc = check_span(N, vis_start, vis_len, vis_len_uniform, Nv_cap);
    if (rc != VITCOP_OK) return rc;
    if (d % 8 || stride_b % 8 || stride_h % 8 || stride_n % 8 || !aligned16(K)) return VITCOP_ERR_UNSUPPORTED;
    if (B > 65535) return VITCOP_ERR_UNSUPPORTED;
    return launch_knorm(K, B, H, d, stride_b, stride_h, stride_n, vis_start, vis_len, vis_len_uniform, score, Nv_cap,
                        static_cast<cudaStream_t>(stream));
}

int vitcop_select(const float* score, const int32_t* label, int B, const int32_t* vis_len, int vis_len_uniform,
                  int Nv_cap, const vitcop_select_params* p, int32_t* keep_idx, int keep_stride, int32_t* n_keep,
                  uint8_t* keep_mask, void* workspace, size_t workspace_bytes, void* stream) {
    if (!score || !p || !keep_idx || !n_keep || B < 0 || Nv_cap < 0 || keep_stride < 0) return VITCOP_ERR_INVALID_ARG;
    if (p->mode != 0 && p->mode != 1) return VITCOP_ERR_INVALID_ARG;
    if (p->budget < 0) return VITCOP_ERR_INVALID_ARG;
    if (p->mode == 1 && !label) return VITCOP_ERR_INVALID_ARG;
    if (!vis_len && (vis_len_uniform < 0 || vis_len_uniform > Nv_cap)) return VITCOP_ERR_INVALID_ARG;
    if (keep_stride < (p->budget < Nv_cap ? p->budget : Nv_cap)) return VITCOP_ERR_INVALID_ARG;
    if (Nv_cap > VITCOP_MAX_VISUAL_TOKENS) return VITCOP_ERR_UNSUPPORTED;
    if (!workspace || workspace_bytes < kStatusBytes) return VITCOP_ERR_WORKSPACE;
    if (!aligned256(workspace)) return VITCOP_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int rc = reset_status(workspace, s);
    if (rc != VITCOP_OK) return rc;
    return launch_select(score, label, B, vis_len, vis_len_uniform, Nv_cap, p->mode, p->largest ? 1 : 0, p->budget,
                         keep_idx, keep_stride, n_keep, keep_mask, static_cast<int*>(workspace), s, false);
}

static int check_compact_args(const void* hidden, const void* K, const void* V, int B, int H, int N, int d, int Dh,
                              int vis_start, const int32_t* vis_len, int vis_len_uniform, void* hidden_out,
                              void* K_out, void* V_out, int Ncap) {
    if (B < 0 || H < 0 || N < 0 || d < 0 || Dh < 0 || Ncap < 0) return VITCOP_ERR_INVALID_ARG;
    if ((hidden == nullptr) != (hidden_out == nullptr)) return VITCOP_ERR_INVALID_ARG;
    if ((K == nullptr) != (K_out == nullptr)) return VITCOP_ERR_INVALID_ARG;
    if ((V == nullptr) != (V_out == nullptr)) return VITCOP_ERR_INVALID_ARG;
    int rc = check_span(N, vis_start, vis_len, vis_len_uniform, -1);
    if (rc != VITCOP_OK) return rc;
    if (d % 8 || Dh % 8) return VITCOP_ERR_UNSUPPORTED;
    if (!aligned16(hidden) || !aligned16(K) || !aligned16(V) || !aligned16(hidden_out) || !aligned16(K_out) ||
        !aligned16(V_out))
        return VITCOP_ERR_UNSUPPORTED;
    if (B > 65535) return VITCOP_ERR_UNSUPPORTED;
    const size_t hin = (size_t)B * N * Dh * 2, hout = (size_t)B * Ncap * Dh * 2;
    const size_t kin = (size_t)B * H * N * d * 2, kout = (size_t)B * H * Ncap * d * 2;
    const void* ins[3] = {hidden, K, V};
    const size_t insz[3] = {hin, kin, kin};
    const void* outs[3] = {hidden_out, K_out, V_out};
    const size_t outsz[3] = {hout, kout, kout};
    for (int i = 0; i < 3; ++i)
        for (int j = 0; j < 3; ++j)
            if (overlaps(ins[i], insz[i], outs[j], outsz[j])) return VITCOP_ERR_INVALID_ARG;
    return VITCOP_OK;
}

int vitcop_compact_kv(const void* hidden, const void* K, const void* V, int B, int H, int N, int d, int Dh,
                      const int32_t* seq_len, int vis_start, const int32_t* vis_len, int vis_len_uniform,
                      const int32_t* keep_idx, int keep_stride, const int32_t* n_keep, void* hidden_out, void* K_out,
                      void* V_out, int Ncap, int32_t* kept_pos, int32_t* out_len, void* stream) {
    if (!keep_idx || !n_keep || !out_len || keep_stride < 0) return VITCOP_ERR_INVALID_ARG;
    int rc = check_compact_args(hidden, K, V, B, H, N, d, Dh, vis_start, vis_len, vis_len_uniform, hidden_out, K_out,
                                V_out, Ncap);
    if (rc != VITCOP_OK) return rc;
    return launch_compact(hidden, K, V, B, H, N, d, Dh, seq_len, vis_start, vis_len, vis_len_uniform, keep_idx,
                          keep_stride, n_keep, hidden_out, K_out, V_out, Ncap, kept_pos, out_len,
                          static_cast<cudaStream_t>(stream), false);
}

int vitcop_prune_step(const void* hidden, const void* K, const void* V, int B, int H, int N, int d, int Dh,
                      const int32_t* seq_len, int vis_start, const int32_t* vis_len, int vis_len_uniform, int Nv_cap,
                      const int32_t* label, int budget, void* hidden_out, void* K_out, void* V_out, int Ncap,
                      int32_t* kept_pos, int32_t* out_len, float* score_out, int32_t* keep_idx_out,
                      int32_t* n_keep_out, void* workspace, size_t workspace_bytes, void* stream) {
    if (!K || !out_len || budget < 0 || Nv_cap < 0) return VITCOP_ERR_INVALID_ARG;
    int rc = check_compact_args(hidden, K, V, B, H, N, d, Dh, vis_start, vis_len, vis_len_uniform, hidden_out, K_out,
                                V_out, Ncap);
    if (rc != VITCOP_OK) return rc;
    rc = check_span(N, vis_start, vis_len, vis_len_uniform, Nv_cap);
    if (rc != VITCOP_OK) return rc;
    if (Nv_cap > VITCOP_MAX_VISUAL_TOKENS) return VITCOP_ERR_UNSUPPORTED;
    const StepWs lay(B, Nv_cap);
    if (!workspace || workspace_bytes < lay.total || !aligned256(workspace)) return VITCOP_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    char* ws = static_cast<char*>(workspace);
    float* score = score_out ? score_out : reinterpret_cast<float*>(ws + lay.off_score);
    int32_t* keep = keep_idx_out ? keep_idx_out : reinterpret_cast<int32_t*>(ws + lay.off_keep);
    int32_t* nkeep = n_keep_out ? n_keep_out : reinterpret_cast<int32_t*>(ws + lay.off_nkeep);
    rc = reset_status(workspace, s);
    if (rc != VITCOP_OK) return rc;
    bool have_knorm = false;
    rc = launch_knorm(K, B, H, d, (int64_t)H * N * d, (int64_t)N * d, d, vis_start, vis_len, vis_len_uniform, score,
                      Nv_cap, s, false, &have_knorm);
    if (rc != VITCOP_OK) return rc;
    // The selection releases its dependents before it waits for its predecessor, and the compaction copies the rows
    // in front of the span before its own wait: that is safe only behind a kernel of this call that has itself
    // waited for everything queued before the call.  With an empty span there is no such kernel, so the selection
    // is then launched in plain stream order.
    rc = launch_select(score, label, B, vis_len, vis_len_uniform, Nv_cap, label ? 1 : 0, 0, budget, keep, Nv_cap,
                       nkeep, nullptr, reinterpret_cast<int*>(ws), s, have_knorm);
    if (rc != VITCOP_OK) return rc;
    return launch_compact(hidden, K, V, B, H, N, d, Dh, seq_len, vis_start, vis_len, vis_len_uniform, keep, Nv_cap,
                          nkeep, hidden_out, K_out, V_out, Ncap, kept_pos, out_len, s, true);
}

int vitcop_collaborative_step(const void* feat, const float* pos, int D, const vitcop_filter_params* fp,
                              const void* hidden, const void* K, const void* V, int B, int H, int N, int d, int Dh,
                              int vis_start, int Nv, int budget, void* hidden_out, void* K_out, void* V_out, int Ncap,
                              int32_t* kept_pos, int32_t* out_len, int32_t* label_out, int32_t* n_clusters_out,
                              float* rho_out, float* delta2_out, int32_t* parent_out, float* score_out,
                              int32_t* keep_idx_out, int32_t* n_keep_out, void* workspace, size_t workspace_bytes,
                              void* stream) {
    if (!feat || !fp || !K || !out_len || !label_out || !n_clusters_out || budget < 0 || Nv < 0 || D < 0)
        return VITCOP_ERR_INVALID_ARG;
    if (fp->metric != 0 && fp->metric != 1) return VITCOP_ERR_INVALID_ARG;
    if (!(fp->d_c > 0.f)) return VITCOP_ERR_INVALID_ARG;
    int rc = check_compact_args(hidden, K, V, B, H, N, d, Dh, vis_start, nullptr, Nv, hidden_out, K_out, V_out, Ncap);
    if (rc != VITCOP_OK) return rc;
    rc = check_span(N, vis_start, nullptr, Nv, Nv);
    if (rc != VITCOP_OK) return rc;
    if (D % 64 || !aligned16(feat) || !aligned8(pos) || Nv > VITCOP_MAX_VISUAL_TOKENS || B > 65535)
        return VITCOP_ERR_UNSUPPORTED;
    const size_t filter_bytes = align_up(filter_workspace_bytes(B, Nv, D), 256);
    const StepWs lay(B, Nv);
    if (!workspace || workspace_bytes < filter_bytes + lay.total || !aligned256(workspace)) return VITCOP_ERR_WORKSPACE;
    int nc = fp->n_centers;
    if (nc <= 0) {
        const double v = std::ceil((double)Nv * fp->alpha);
        nc = v < 0 ? 0 : (v > Nv ? Nv : (int)v);
    }
    if (nc > Nv) nc = Nv;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    char* ws = static_cast<char*>(workspace);
    char* ws2 = ws + filter_bytes;
    float* score = score_out ? score_out : reinterpret_cast<float*>(ws2 + lay.off_score);
    int32_t* keep = keep_idx_out ? keep_idx_out : reinterpret_cast<int32_t*>(ws2 + lay.off_keep);
    int32_t* nkeep = n_keep_out ? n_keep_out : reinterpret_cast<int32_t*>(ws2 + lay.off_nkeep);
    rc = record_cuda(cudaMemsetAsync(workspace, 0, filter_zeroed_bytes(B, Nv), s));
    if (rc != VITCOP_OK) return rc;
    if (B == 0) return VITCOP_OK;
    if (Nv > 0) {
        const KnormJob job = {K, B, H, N, d, vis_start, Nv, score};
        rc = launch_filter(feat, pos, B, Nv, D, *fp, nc, label_out, n_clusters_out, rho_out, delta2_out, parent_out,
                           workspace, s, &job);
        if (rc != VITCOP_OK) return rc;
    }
    // (plain stream order when the filter was skipped: see vitcop_prune_step)
    rc = launch_select(score, label_out, B, nullptr, Nv, Nv, 1, 0, budget, keep, Nv, nkeep, nullptr,
                       reinterpret_cast<int*>(ws), s, Nv > 0);
    if (rc != VITCOP_OK) return rc;
    return launch_compact(hidden, K, V, B, H, N, d, Dh, nullptr, vis_start, nullptr, Nv, keep, Nv, nkeep, hidden_out,
                          K_out, V_out, Ncap, kept_pos, out_len, s, true);
}

int vitcop_merge_clusters(const void* hidden, int B, int N, int Dh, int vis_start, const int32_t* vis_len,
                          int vis_len_uniform, int Nv_cap, const int32_t* label, const uint8_t* keep_mask, void* merged,
                          float* merged_f32, int32_t* merged_label, int32_t* merged_count, int32_t* n_merged, int Mcap,
                          void* workspace, size_t workspace_bytes, void* stream) {
    if (!hidden || !label || !keep_mask || !merged_label || !merged_count || !n_merged) return VITCOP_ERR_INVALID_ARG;
    if (B < 0 || N < 0 || Dh < 0 || Nv_cap < 0 || Mcap < 0) return VITCOP_ERR_INVALID_ARG;
    int rc = check_span(N, vis_start, vis_len, vis_len_uniform, Nv_cap);
    if (rc != VITCOP_OK) return rc;
    if (Dh % 8 || !aligned16(hidden) || !aligned16(merged) || !aligned16(merged_f32)) return VITCOP_ERR_UNSUPPORTED;
    if (Nv_cap > VITCOP_MAX_VISUAL_TOKENS || B > 65535) return VITCOP_ERR_UNSUPPORTED;
    if (!workspace || workspace_bytes < merge_workspace_bytes(B, Nv_cap, Mcap) || !aligned256(workspace))
        return VITCOP_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    rc = reset_status(workspace, s);
    if (rc != VITCOP_OK) return rc;
    return launch_merge(hidden, B, N, Dh, vis_start, vis_len, vis_len_uniform, Nv_cap, label, keep_mask, merged,
                        merged_f32, merged_label, merged_count, n_merged, Mcap, workspace, s);
}

int vitcop_cls_saliency(const void* q_cls, const void* K, int B, int H, int M, int d, float scale, float* saliency,
                        float* cls_self, void* workspace, size_t workspace_bytes, void* stream) {
    if (!q_cls || !K || (!saliency && M > 1) || B < 0 || H < 0 || M < 0 || d < 0) return VITCOP_ERR_INVALID_ARG;
    if (d % 8 || !aligned16(q_cls) || !aligned16(K) || B > 65535 || H > 4096 || d > 4096) return VITCOP_ERR_UNSUPPORTED;
    if (!workspace || workspace_bytes < saliency_workspace_bytes(B, H, M) || !aligned256(workspace))
        return VITCOP_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int rc = reset_status(workspace, s);
    if (rc != VITCOP_OK) return rc;
    return launch_cls_saliency(q_cls, K, B, H, M, d, scale, saliency, cls_self, workspace, s);
}

int vitcop_kproj_knorm(const void* hidden, const void* W_k, int B, int N, int Dh, int H, int d, const float* rope_cos,
                       const float* rope_sin, const int32_t* position_ids, int n_pos, void* K_out, int vis_start, int Nv,
                       float* score, void* workspace, size_t workspace_bytes, void* stream) {
    if (!hidden || !W_k || !K_out || B < 0 || N < 0 || Dh < 0 || H < 0 || d < 0 || Nv < 0 || vis_start < 0)
        return VITCOP_ERR_INVALID_ARG;
    if ((rope_cos == nullptr) != (rope_sin == nullptr)) return VITCOP_ERR_INVALID_ARG;
    if (rope_cos && n_pos <= 0) return VITCOP_ERR_INVALID_ARG;
    if (score && vis_start + (int64_t)Nv > N) return VITCOP_ERR_INVALID_ARG;
    if (Dh % 64 || d % 32 || !aligned16(hidden) || !aligned16(W_k) || !aligned16(K_out)) return VITCOP_ERR_UNSUPPORTED;
    if (rope_cos && ((d != 64 && d != 128 && d != 256) || !aligned16(rope_cos) || !aligned16(rope_sin)))
        return VITCOP_ERR_UNSUPPORTED;
    if ((int64_t)B * N > 0x7fffffff || (int64_t)H * d > 0x7fffffff || B > 65535) return VITCOP_ERR_UNSUPPORTED;
    if (!workspace || workspace_bytes < kproj_workspace_bytes(B, N, H, d) || !aligned256(workspace))
        return VITCOP_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int rc = reset_status(workspace, s);
    if (rc != VITCOP_OK) return rc;
    if (B == 0 || N == 0 || H == 0 || d == 0 || Dh == 0) return VITCOP_OK;
    return launch_kproj_knorm(hidden, W_k, B, N, Dh, H, d, rope_cos, rope_sin, position_ids, n_pos, K_out, vis_start,
                              score ? Nv : 0, score, workspace, s);
}

int vitcop_prune_step_static(const void* hidden, const void* K, const void* V, int B, int H, int N, int d, int Dh,
                             const int32_t* seq_len, int vis_start, const int32_t* vis_len, int vis_len_uniform,
                             int Nv_cap, const int32_t* label, int budget, void* hidden_out, void* K_out, void* V_out,
                             int Ncap, int32_t* kept_pos, int32_t* out_len, float* score_out, int32_t* keep_idx_out,
                             int32_t* n_keep_out, void* stream) {
    if (B < 0 || Nv_cap < 0) return VITCOP_ERR_INVALID_ARG;
    if (StepWs(B, Nv_cap).total > kStaticScratchBytes) return VITCOP_ERR_UNSUPPORTED;
    void* scratch = nullptr;
    const int rc = static_scratch_address(&scratch);
    if (rc != VITCOP_OK) return rc;
    return vitcop_prune_step(hidden, K, V, B, H, N, d, Dh, seq_len, vis_start, vis_len, vis_len_uniform, Nv_cap, label,
                             budget, hidden_out, K_out, V_out, Ncap, kept_pos, out_len, score_out, keep_idx_out,
                             n_keep_out, scratch, kStaticScratchBytes, stream);
}

int vitcop_redundancy_filter(const void* feat, const float* pos, int B, int n, int D, const vitcop_filter_params* p,
                             int32_t* label, int32_t* n_clusters, float* rho, float* delta2, int32_t* parent,
                             void* workspace, size_t workspace_bytes, void* stream) {
    if (!feat || !p || !label || !n_clusters || B < 0 || n < 0 || D < 0) return VITCOP_ERR_INVALID_ARG;
    if (p->metric != 0 && p->metric != 1) return VITCOP_ERR_INVALID_ARG;
    if (!(p->d_c > 0.f)) return VITCOP_ERR_INVALID_ARG;
    if (D % 64 || !aligned16(feat) || !aligned8(pos) || n > VITCOP_MAX_VISUAL_TOKENS || B > 65535)
        return VITCOP_ERR_UNSUPPORTED;
    if (!workspace || workspace_bytes < filter_workspace_bytes(B, n, D) || !aligned256(workspace))
        return VITCOP_ERR_WORKSPACE;
    int nc = p->n_centers;
    if (nc <= 0) {
        const double v = std::ceil((double)n * p->alpha);
        nc = v < 0 ? 0 : (v > n ? n : (int)v);
    }
    if (nc > n) nc = n;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int rc = record_cuda(cudaMemsetAsync(workspace, 0, filter_zeroed_bytes(B, n), s));
    if (rc != VITCOP_OK) return rc;
    if (B == 0 || n == 0) return VITCOP_OK;
    return launch_filter(feat, pos, B, n, D, *p, nc, label, n_clusters, rho, delta2, parent, workspace, s);
}

int vitcop_similarity_rows(const void* feat, int B, int n, int D, int metric, int row_begin, int row_end, float* out,
                           void* workspace, size_t workspace_bytes, void* stream) {
    if (!feat || !out || B < 0 || n < 0 || D < 0) return VITCOP_ERR_INVALID_ARG;
    if (metric != 0 && metric != 1) return VITCOP_ERR_INVALID_ARG;
    if (row_begin < 0 || row_end < row_begin || row_end > n) return VITCOP_ERR_INVALID_ARG;
    if (D % 64 || !aligned16(feat) || n > VITCOP_MAX_VISUAL_TOKENS || B > 65535)
        return VITCOP_ERR_UNSUPPORTED;
    if (!workspace || workspace_bytes < similarity_workspace_bytes(B, n, D) || !aligned256(workspace))
        return VITCOP_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int rc = reset_status(workspace, s);
    if (rc != VITCOP_OK) return rc;
    if (B == 0 || n == 0 || row_end == row_begin) return VITCOP_OK;
    return launch_similarity_rows(feat, B, n, D, metric, row_begin, row_end, out, workspace, s);
}

}  // extern "C"
