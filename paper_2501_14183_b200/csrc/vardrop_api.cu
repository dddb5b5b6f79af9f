// C ABI of the library: argument checks, workspace carving, status text.  All arithmetic lives in the
// kernel translation units; nothing here allocates device memory or synchronises.
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <utility>
#include <vector>

#include "common.cuh"
#include "kernels.h"

namespace vardrop {

static thread_local char g_last_error[512] = "";

int fail(int status, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_last_error, sizeof(g_last_error), fmt, ap);
    va_end(ap);
    return status;
}

int check_cuda(cudaError_t e, const char* what) {
    if (e == cudaSuccess) return VARDROP_OK;
    return fail(VARDROP_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

static int check_ptr(const void* p, const char* name, bool required) {
    if (!p) return required ? fail(VARDROP_ERR_INVALID_ARG, "%s is NULL", name) : VARDROP_OK;
    if (!aligned16(p)) return fail(VARDROP_ERR_INVALID_ARG, "%s is not 16-byte aligned", name);
    return VARDROP_OK;
}

static int check_ws(const void* ws, size_t have, size_t need) {
    if (int st = check_ptr(ws, "ws", true)) return st;
    if (have < need) return fail(VARDROP_ERR_WORKSPACE, "workspace of %zu bytes given, %zu needed", have, need);
    return VARDROP_OK;
}

// ---- launch counter and optional per-kernel event timer ---------------------------------------------------
namespace {
std::mutex g_prof_mutex;
bool g_prof_on = false;
long long g_launches = 0;
std::vector<std::pair<cudaEvent_t, cudaEvent_t>> g_prof_events[K_COUNT];   // pairs recorded since the timer was armed
std::vector<std::pair<cudaEvent_t, cudaEvent_t>> g_prof_free;              // pairs ready for reuse
const char* const g_kernel_names[K_COUNT] = {"hash_kernel", "select_small_kernel", "select_count_kernel", "select_group_kernel", "select_sample_kernel", "gather_kernel",
                                             "attn_fwd_kernel", "bwd_prep_kernel", "attn_bwd_kernel", "bwd_convert_kernel", "pearson_normalize_kernel",
                                             "pearson_max_kernel", "gather_rows_kernel"};
}  // namespace

LaunchScope::LaunchScope(int id, cudaStream_t stream) : id_(id), stream_(stream), stop_(nullptr) {
    std::lock_guard<std::mutex> lock(g_prof_mutex);
    ++g_launches;
    if (!g_prof_on) return;
    std::pair<cudaEvent_t, cudaEvent_t> ev;
    if (!g_prof_free.empty()) {
        ev = g_prof_free.back();
        g_prof_free.pop_back();
    } else if (cudaEventCreate(&ev.first) != cudaSuccess || cudaEventCreate(&ev.second) != cudaSuccess) {
        return;
    }
    cudaEventRecord(ev.first, stream);
    g_prof_events[id].push_back(ev);
    stop_ = ev.second;
}

LaunchScope::~LaunchScope() {
    if (stop_) cudaEventRecord(static_cast<cudaEvent_t>(stop_), stream_);
}

// A wait that nothing ever completes: one warp polls a fresh barrier with the library's bounded wait and a caller-chosen limit,
// then reports the way every kernel of the library does (status word, normal exit).
__global__ void bounded_wait_probe_kernel(int* status, unsigned long long limit_ns) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        mbar_fence_init();
    }
    __syncthreads();
    chain_wait();
    chain_release();
    const bool done = mbar_wait(&bar, 0, limit_ns);
    if (!__all_sync(0xffffffffu, done) && threadIdx.x == 0) set_status(status, VARDROP_ERR_TIMEOUT);
}

}  // namespace vardrop

using namespace vardrop;

#define VD_CHECK(expr) do { if (int st_ = (expr)) return st_; } while (0)

extern "C" {

const char* vardrop_status_string(int status) {
    switch (status) {
        case VARDROP_OK: return "ok";
        case VARDROP_ERR_INVALID_ARG: return "invalid argument";
        case VARDROP_ERR_UNSUPPORTED: return "unsupported shape";
        case VARDROP_ERR_WORKSPACE: return "workspace too small";
        case VARDROP_ERR_CUDA: return "CUDA error";
        case VARDROP_ERR_TIMEOUT: return "bounded device wait timed out";
        case VARDROP_ERR_NONFINITE: return "non-finite amplitude";
        default: return "unknown status";
    }
}

const char* vardrop_last_error(void) { return g_last_error; }
const char* vardrop_version(void) { return "0.1"; }

int vardrop_ws_status(const void* ws, void* stream) {
    if (!ws) return fail(VARDROP_ERR_INVALID_ARG, "ws is NULL");
    int word = 0;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (int st = check_cuda(cudaMemcpyAsync(&word, ws, sizeof(int), cudaMemcpyDeviceToHost, s), "ws_status: copy")) return st;
    if (int st = check_cuda(cudaStreamSynchronize(s), "ws_status: synchronize")) return st;
    return word;
}

int vardrop_probe_bounded_wait(void* ws, size_t ws_bytes, unsigned int limit_us, void* stream) {
    VD_CHECK(check_ws(ws, ws_bytes, kWsHeaderBytes));
    if (limit_us < 1 || limit_us > 100000) return fail(VARDROP_ERR_INVALID_ARG, "probe: limit of %u us outside 1..100000", limit_us);
    const cudaError_t err = launch_chained(bounded_wait_probe_kernel, dim3(1), dim3(32), 0, static_cast<cudaStream_t>(stream), static_cast<int*>(ws),
                                           static_cast<unsigned long long>(limit_us) * 1000ull);
    return check_cuda(err, "probe: launch");
}

long long vardrop_launch_count(void) {
    std::lock_guard<std::mutex> lock(g_prof_mutex);
    return g_launches;
}

int vardrop_profile_kernels(void) { return K_COUNT; }

const char* vardrop_profile_kernel_name(int id) { return id >= 0 && id < K_COUNT ? g_kernel_names[id] : ""; }

int vardrop_profile_enable(int on) {
    std::lock_guard<std::mutex> lock(g_prof_mutex);
    for (int id = 0; id < K_COUNT; ++id) {
        for (auto& ev : g_prof_events[id]) g_prof_free.push_back(ev);
        g_prof_events[id].clear();
    }
    g_prof_on = on != 0;
    return VARDROP_OK;
}

int vardrop_profile_read(int id, double* total_ms, long long* launches) {
    if (id < 0 || id >= K_COUNT || !total_ms || !launches) return fail(VARDROP_ERR_INVALID_ARG, "profile_read: bad argument");
    std::lock_guard<std::mutex> lock(g_prof_mutex);
    double sum = 0.0;
    for (auto& ev : g_prof_events[id]) {
        if (int st = check_cuda(cudaEventSynchronize(ev.second), "profile_read: event synchronize")) return st;
        float ms = 0.f;
        if (int st = check_cuda(cudaEventElapsedTime(&ms, ev.first, ev.second), "profile_read: elapsed time")) return st;
        sum += ms;
    }
    *total_ms = sum;
    *launches = static_cast<long long>(g_prof_events[id].size());
    return VARDROP_OK;
}

size_t vardrop_hash_workspace_bytes(const vardrop_hash_cfg* cfg) { return cfg ? hash_workspace_bytes(*cfg) : 0; }

int vardrop_hash(const float* x, const vardrop_hash_cfg* cfg, uint64_t* keys, int32_t* freqs, float* amp_dbg, void* ws,
                 size_t ws_bytes, void* stream) {
    if (!cfg) return fail(VARDROP_ERR_INVALID_ARG, "cfg is NULL");
    int f_lo, f_hi;
    VD_CHECK(hash_validate(*cfg, &f_lo, &f_hi));
    VD_CHECK(check_ptr(x, "x", true));
    VD_CHECK(check_ptr(keys, "keys", true));
    VD_CHECK(check_ptr(freqs, "freqs", false));
    VD_CHECK(check_ptr(amp_dbg, "amp_dbg", false));
    VD_CHECK(check_ws(ws, ws_bytes, hash_workspace_bytes(*cfg)));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    return hash_launch(x, *cfg, keys, freqs, amp_dbg, static_cast<int*>(ws), s);
}

size_t vardrop_select_workspace_bytes(const vardrop_select_cfg* cfg) {
    if (!cfg || select_validate(*cfg) != VARDROP_OK) return 0;
    return select_workspace_bytes(*cfg);
}

int vardrop_select(const uint64_t* keys, const vardrop_select_cfg* cfg, int32_t* group_id, int32_t* group_offsets,
                   int32_t* members, int32_t* n_groups, int32_t* sel_idx, int32_t* n_sel, int32_t* inv_idx, void* ws,
                   size_t ws_bytes, void* stream) {
    if (!cfg) return fail(VARDROP_ERR_INVALID_ARG, "cfg is NULL");
    VD_CHECK(select_validate(*cfg));
    VD_CHECK(check_ptr(keys, "keys", true));
    VD_CHECK(check_ptr(group_id, "group_id", true));
    VD_CHECK(check_ptr(group_offsets, "group_offsets", true));
    VD_CHECK(check_ptr(members, "members", true));
    VD_CHECK(check_ptr(n_groups, "n_groups", true));
    VD_CHECK(check_ptr(sel_idx, "sel_idx", true));
    VD_CHECK(check_ptr(n_sel, "n_sel", true));
    VD_CHECK(check_ptr(inv_idx, "inv_idx", true));
    VD_CHECK(check_ws(ws, ws_bytes, select_workspace_bytes(*cfg)));
    return select_launch(keys, *cfg, group_id, group_offsets, members, n_groups, sel_idx, n_sel, inv_idx, ws,
                         static_cast<cudaStream_t>(stream));
}

int vardrop_select_static(const uint64_t* keys, const vardrop_select_cfg* cfg, int32_t* group_id, int32_t* group_offsets,
                          int32_t* members, int32_t* n_groups, int32_t* sel_idx, int32_t* n_sel, int32_t* inv_idx, void* stream) {
    if (!cfg) return fail(VARDROP_ERR_INVALID_ARG, "cfg is NULL");
    VD_CHECK(select_validate(*cfg));
    VD_CHECK(check_ptr(keys, "keys", true));
    VD_CHECK(check_ptr(group_id, "group_id", true));
    VD_CHECK(check_ptr(group_offsets, "group_offsets", true));
    VD_CHECK(check_ptr(members, "members", true));
    VD_CHECK(check_ptr(n_groups, "n_groups", true));
    VD_CHECK(check_ptr(sel_idx, "sel_idx", true));
    VD_CHECK(check_ptr(n_sel, "n_sel", true));
    VD_CHECK(check_ptr(inv_idx, "inv_idx", true));
    return select_static_launch(keys, *cfg, group_id, group_offsets, members, n_groups, sel_idx, n_sel, inv_idx,
                                static_cast<cudaStream_t>(stream));
}

int vardrop_gather_rows(const float* x, const int32_t* sel_idx, const int32_t* n_sel, const vardrop_gather_cfg* cfg, float* x_sel, void* stream) {
    if (!cfg) return fail(VARDROP_ERR_INVALID_ARG, "cfg is NULL");
    VD_CHECK(gather_rows_validate(*cfg));
    VD_CHECK(check_ptr(x, "x", true));
    VD_CHECK(check_ptr(sel_idx, "sel_idx", true));
    VD_CHECK(check_ptr(n_sel, "n_sel", true));
    VD_CHECK(check_ptr(x_sel, "x_sel", true));
    return gather_rows_launch(x, sel_idx, n_sel, *cfg, x_sel, static_cast<cudaStream_t>(stream));
}

size_t vardrop_attn_workspace_bytes(const vardrop_attn_cfg* cfg) {
    if (!cfg || attn_validate(*cfg) != VARDROP_OK) return 0;
    return attn_workspace_bytes(*cfg);
}

int vardrop_attn_fwd(const void* q, const void* k, const void* v, const int32_t* sel_idx, const int32_t* n_sel,
                     const vardrop_attn_cfg* cfg, void* o, float* lse, void* ws, size_t ws_bytes, void* stream) {
    if (!cfg) return fail(VARDROP_ERR_INVALID_ARG, "cfg is NULL");
    VD_CHECK(attn_validate(*cfg));
    VD_CHECK(check_ptr(q, "q", true));
    VD_CHECK(check_ptr(k, "k", true));
    VD_CHECK(check_ptr(v, "v", true));
    VD_CHECK(check_ptr(sel_idx, "sel_idx", false));
    if (sel_idx) VD_CHECK(check_ptr(n_sel, "n_sel", true));
    VD_CHECK(check_ptr(o, "o", true));
    VD_CHECK(check_ptr(lse, "lse", true));
    VD_CHECK(check_ws(ws, ws_bytes, attn_workspace_bytes(*cfg)));
    return attn_fwd_launch(q, k, v, sel_idx, n_sel, *cfg, o, lse, ws, static_cast<cudaStream_t>(stream));
}

int vardrop_attn_bwd(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* d_o,
                     const int32_t* sel_idx, const int32_t* n_sel, const int32_t* inv_idx, const vardrop_attn_cfg* cfg,
                     void* dq, void* dk, void* dv, void* ws, size_t ws_bytes, void* stream) {
    if (!cfg) return fail(VARDROP_ERR_INVALID_ARG, "cfg is NULL");
    VD_CHECK(attn_validate(*cfg));
    VD_CHECK(check_ptr(q, "q", true));
    VD_CHECK(check_ptr(k, "k", true));
    VD_CHECK(check_ptr(v, "v", true));
    VD_CHECK(check_ptr(o, "o", true));
    VD_CHECK(check_ptr(lse, "lse", true));
    VD_CHECK(check_ptr(d_o, "d_o", true));
    VD_CHECK(check_ptr(sel_idx, "sel_idx", false));
    if (sel_idx) {
        VD_CHECK(check_ptr(n_sel, "n_sel", true));
        VD_CHECK(check_ptr(inv_idx, "inv_idx", true));
    }
    VD_CHECK(check_ptr(dq, "dq", true));
    VD_CHECK(check_ptr(dk, "dk", true));
    VD_CHECK(check_ptr(dv, "dv", true));
    VD_CHECK(check_ws(ws, ws_bytes, attn_workspace_bytes(*cfg)));
    return attn_bwd_launch(q, k, v, o, lse, d_o, sel_idx, n_sel, inv_idx, *cfg, dq, dk, dv, ws, static_cast<cudaStream_t>(stream));
}

size_t vardrop_pearson_workspace_bytes(const vardrop_pearson_cfg* cfg) {
    if (!cfg || pearson_validate(*cfg) != VARDROP_OK) return 0;
    return pearson_workspace_bytes(*cfg);
}

int vardrop_pearson_max(const float* x, const vardrop_pearson_cfg* cfg, float* max_rho, int32_t* n_above, void* ws, size_t ws_bytes,
                        void* stream) {
    if (!cfg) return fail(VARDROP_ERR_INVALID_ARG, "cfg is NULL");
    VD_CHECK(pearson_validate(*cfg));
    VD_CHECK(check_ptr(x, "x", true));
    VD_CHECK(check_ptr(max_rho, "max_rho", true));
    VD_CHECK(check_ptr(n_above, "n_above", true));
    VD_CHECK(check_ws(ws, ws_bytes, pearson_workspace_bytes(*cfg)));
    return pearson_launch(x, *cfg, max_rho, n_above, ws, static_cast<cudaStream_t>(stream));
}

}  // extern "C"
