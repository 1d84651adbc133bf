// C ABI of libgar: argument validation, workspace handling and the enqueue of
// the three kernels (distances -> selection -> coordinate phase).
#include <cstdio>
#include <mutex>

#include "gar_internal.cuh"

namespace {

using gar::Workspace;

constexpr int kMaxDevices = 64;

struct DeviceState {
    bool    known = false;
    int     sm_count = 0;
    char*   workspace = nullptr;          // cached workspace (gar_aggregate, NULL workspace)
    // host-path staging
    float*  stage_grads = nullptr;
    size_t  stage_grads_elems = 0;
    float*  stage_out = nullptr;
    size_t  stage_out_elems = 0;
    cudaStream_t copy_stream = nullptr, compute_stream = nullptr;
    cudaEvent_t  slab_ready[2] = {nullptr, nullptr};
    cudaEvent_t  computed = nullptr;
};

DeviceState g_dev[kMaxDevices];
std::mutex  g_mutex;

bool rule_ok(int rule) { return rule >= GAR_AVERAGE && rule <= GAR_MULTI_BULYAN; }

int precondition(int rule, int n, int f) {
    if (rule == GAR_KRUM || rule == GAR_MULTI_KRUM) return n >= 2 * f + 3;
    if (rule == GAR_BULYAN || rule == GAR_MULTI_BULYAN) return n >= 4 * f + 3;
    return 1;
}

int default_theta(int rule, int n, int f) {
    switch (rule) {
        case GAR_MEDIAN:       return n;
        case GAR_BULYAN:       return n - 2 * f;
        case GAR_MULTI_BULYAN: return n - 2 * f - 2;
        default:               return 1;
    }
}

int beta_for(int rule, int theta, int f) {
    if (rule == GAR_BULYAN || rule == GAR_MULTI_BULYAN) return theta - 2 * f;
    return 1;
}

int basic_checks(int rule, int n, int f, int64_t d) {
    if (!rule_ok(rule) || n < 1 || f < 0 || d < 1) return GAR_ERR_INVALID_ARG;
    if (n > GAR_MAX_N) return GAR_ERR_UNSUPPORTED;
    if (!precondition(rule, n, f)) return GAR_ERR_PRECONDITION;
    return GAR_OK;
}

// Current device's state; creates the cached pieces that were asked for.
int device_state(DeviceState** out, bool need_workspace) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return GAR_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return GAR_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceState& st = g_dev[dev];
    if (!st.known) {
        if (cudaDeviceGetAttribute(&st.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
            return GAR_ERR_CUDA;
        st.known = true;
    }
    if (need_workspace && !st.workspace) {
        if (cudaMalloc(&st.workspace, gar::kWorkspaceBytes) != cudaSuccess) return GAR_ERR_CUDA;
        if (cudaMemset(st.workspace, 0, gar::kCtrlBytes) != cudaSuccess) return GAR_ERR_CUDA;
    }
    *out = &st;
    return GAR_OK;
}

int resolve_workspace(void* user_ws, size_t user_bytes, DeviceState** st, Workspace* ws) {
    int rc = device_state(st, user_ws == nullptr);
    if (rc != GAR_OK) return rc;
    if (user_ws) {
        if (reinterpret_cast<uintptr_t>(user_ws) % 256 != 0 || user_bytes < gar::kWorkspaceBytes)
            return GAR_ERR_WORKSPACE;
        ws->base = static_cast<char*>(user_ws);
    } else {
        ws->base = (*st)->workspace;
    }
    return GAR_OK;
}

bool overlaps(const void* a, size_t abytes, const void* b, size_t bbytes) {
    const uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
    return a0 < b0 + bbytes && b0 < a0 + abytes;
}

// Enqueue the whole rule for device buffers.
int enqueue(int rule, const float* grads, int n, int f, int64_t d, int64_t ld, float* out, int m, int theta,
            int median_of_agr, const Workspace& ws, double* dist_out, gar_selection_t* sel_out,
            int sm_count, cudaStream_t stream) {
    const int beta = beta_for(rule, theta, f);
    double* dist = dist_out ? dist_out : ws.dist();
    gar_selection_t* sel = sel_out ? sel_out : ws.selection();
    cudaError_t err;
    const bool needs_dist = !(rule == GAR_AVERAGE || rule == GAR_MEDIAN);
    if (needs_dist) {
        err = gar::launch_distances(grads, n, d, ld, dist, ws, sm_count, stream);
        if (err != cudaSuccess) return GAR_ERR_CUDA;
    }
    err = gar::launch_select(rule, dist, n, f, m, theta, beta, median_of_agr, sel, stream);
    if (err != cudaSuccess) return GAR_ERR_CUDA;
    const int preagg = (rule == GAR_MULTI_BULYAN || rule == GAR_MULTI_KRUM || rule == GAR_AVERAGE) ? 1 : 0;
    err = gar::launch_coordinate(grads, n, d, ld, sel, theta, preagg, out, sm_count, stream);
    if (err != cudaSuccess) return GAR_ERR_CUDA;
    return GAR_OK;
}

}  // namespace

extern "C" {

int gar_version(void) { return GAR_VERSION; }

const char* gar_status_string(int status) {
    switch (status) {
        case GAR_OK:               return "ok";
        case GAR_ERR_INVALID_ARG:  return "invalid argument";
        case GAR_ERR_PRECONDITION: return "precondition violated: need n >= 2f+3 (Krum family) or n >= 4f+3 (Bulyan family)";
        case GAR_ERR_UNSUPPORTED:  return "unsupported: more than 64 gradients";
        case GAR_ERR_WORKSPACE:    return "workspace missing, misaligned or too small";
        case GAR_ERR_CUDA:         return "CUDA runtime or launch error";
        case GAR_ERR_TIMEOUT:      return "device-side wait timed out";
        default:                   return "unknown status";
    }
}

int gar_theta(int rule, int n, int f) {
    if (basic_checks(rule, n, f, 1) != GAR_OK) return -1;
    return default_theta(rule, n, f);
}

int gar_beta(int rule, int n, int f) {
    if (basic_checks(rule, n, f, 1) != GAR_OK) return -1;
    return beta_for(rule, default_theta(rule, n, f), f);
}

size_t gar_workspace_bytes(int rule, int n, int f, int64_t d) {
    if (basic_checks(rule, n, f, d) != GAR_OK) return 0;
    return gar::kWorkspaceBytes;
}

int gar_aggregate_ex(const gar_params_t* p) {
    if (!p) return GAR_ERR_INVALID_ARG;
    int rc = basic_checks(p->rule, p->n, p->f, p->d);
    if (rc != GAR_OK) return rc;
    if (!p->grads || !p->out) return GAR_ERR_INVALID_ARG;
    const int64_t ld = p->ld ? p->ld : p->d;
    if (ld < p->d) return GAR_ERR_INVALID_ARG;
    if (overlaps(p->grads, (size_t(p->n - 1) * ld + p->d) * sizeof(float), p->out, size_t(p->d) * sizeof(float)))
        return GAR_ERR_INVALID_ARG;
    int theta = default_theta(p->rule, p->n, p->f);
    int m = 0;
    if (p->m != 0) {
        if (p->rule != GAR_MULTI_KRUM || p->m < 1 || p->m > p->n - p->f - 2) return GAR_ERR_INVALID_ARG;
        m = p->m;
    }
    if (p->theta != 0) {
        if (p->rule != GAR_MULTI_BULYAN || p->theta < 2 * p->f + 1 || p->theta > p->n - 2 * p->f - 2)
            return GAR_ERR_INVALID_ARG;
        theta = p->theta;
    }
    if (p->median_of_agr != 0 && (p->rule != GAR_MULTI_BULYAN || p->median_of_agr != 1)) return GAR_ERR_INVALID_ARG;
    DeviceState* st = nullptr;
    Workspace ws{};
    rc = resolve_workspace(p->workspace, p->workspace_bytes, &st, &ws);
    if (rc != GAR_OK) return rc;
    return enqueue(p->rule, p->grads, p->n, p->f, p->d, ld, p->out, m, theta, p->median_of_agr, ws, p->dist_out,
                   p->selection_out, st->sm_count, static_cast<cudaStream_t>(p->stream));
}

int gar_aggregate(int rule, const float* grads, int n, int f, int64_t d, float* out, void* stream) {
    gar_params_t p{};
    p.rule = rule; p.n = n; p.f = f; p.d = d; p.ld = d;
    p.grads = grads; p.out = out; p.stream = stream;
    return gar_aggregate_ex(&p);
}

int gar_pairwise_distances(const float* grads, int n, int64_t d, int64_t ld, double* dist, void* workspace,
                           size_t workspace_bytes, void* stream) {
    if (!grads || !dist || n < 1 || d < 1) return GAR_ERR_INVALID_ARG;
    if (n > GAR_MAX_N) return GAR_ERR_UNSUPPORTED;
    if (ld == 0) ld = d;
    if (ld < d) return GAR_ERR_INVALID_ARG;
    DeviceState* st = nullptr;
    Workspace ws{};
    int rc = resolve_workspace(workspace, workspace_bytes, &st, &ws);
    if (rc != GAR_OK) return rc;
    cudaError_t err = gar::launch_distances(grads, n, d, ld, dist, ws, st->sm_count, static_cast<cudaStream_t>(stream));
    return err == cudaSuccess ? GAR_OK : GAR_ERR_CUDA;
}

int gar_select(int rule, const double* dist, int n, int f, int m, int theta, int median_of_agr,
               gar_selection_t* sel, void* stream) {
    int rc = basic_checks(rule, n, f, 1);
    if (rc != GAR_OK) return rc;
    if (!sel) return GAR_ERR_INVALID_ARG;
    const bool needs_dist = !(rule == GAR_AVERAGE || rule == GAR_MEDIAN);
    if (needs_dist && !dist) return GAR_ERR_INVALID_ARG;
    int th = default_theta(rule, n, f);
    if (m != 0 && (rule != GAR_MULTI_KRUM || m < 1 || m > n - f - 2)) return GAR_ERR_INVALID_ARG;
    if (theta != 0) {
        if (rule != GAR_MULTI_BULYAN || theta < 2 * f + 1 || theta > n - 2 * f - 2) return GAR_ERR_INVALID_ARG;
        th = theta;
    }
    if (median_of_agr != 0 && (rule != GAR_MULTI_BULYAN || median_of_agr != 1)) return GAR_ERR_INVALID_ARG;
    cudaError_t err = gar::launch_select(rule, dist, n, f, m, th, beta_for(rule, th, f), median_of_agr, sel,
                                         static_cast<cudaStream_t>(stream));
    return err == cudaSuccess ? GAR_OK : GAR_ERR_CUDA;
}

int gar_schedule_from_tables(gar_selection_t* sel, void* stream) {
    if (!sel) return GAR_ERR_INVALID_ARG;
    cudaError_t err = gar::launch_schedule_only(sel, static_cast<cudaStream_t>(stream));
    return err == cudaSuccess ? GAR_OK : GAR_ERR_CUDA;
}

int gar_coordinate_phase(const float* grads, int n, int64_t d, int64_t ld, const gar_selection_t* sel, int theta,
                         int preagg, float* out, void* stream) {
    if (!grads || !sel || !out || n < 1 || d < 1 || theta < 1 || theta > GAR_MAX_N) return GAR_ERR_INVALID_ARG;
    if (n > GAR_MAX_N) return GAR_ERR_UNSUPPORTED;
    if (ld == 0) ld = d;
    if (ld < d) return GAR_ERR_INVALID_ARG;
    DeviceState* st = nullptr;
    int rc = device_state(&st, false);
    if (rc != GAR_OK) return rc;
    cudaError_t err = gar::launch_coordinate(grads, n, d, ld, sel, theta, preagg ? 1 : 0, out, st->sm_count,
                                             static_cast<cudaStream_t>(stream));
    return err == cudaSuccess ? GAR_OK : GAR_ERR_CUDA;
}

int gar_aggregate_host(int rule, const float* grads, int n, int f, int64_t d, float* out) {
    int rc = basic_checks(rule, n, f, d);
    if (rc != GAR_OK) return rc;
    if (!grads || !out) return GAR_ERR_INVALID_ARG;
    DeviceState* st = nullptr;
    rc = device_state(&st, true);
    if (rc != GAR_OK) return rc;
    // staging buffers and streams (cached, grown on demand)
    const size_t need = size_t(n) * size_t(d);
    if (st->stage_grads_elems < need) {
        if (st->stage_grads) cudaFree(st->stage_grads);
        st->stage_grads = nullptr; st->stage_grads_elems = 0;
        if (cudaMalloc(&st->stage_grads, need * sizeof(float)) != cudaSuccess) return GAR_ERR_CUDA;
        st->stage_grads_elems = need;
    }
    if (st->stage_out_elems < size_t(d)) {
        if (st->stage_out) cudaFree(st->stage_out);
        st->stage_out = nullptr; st->stage_out_elems = 0;
        if (cudaMalloc(&st->stage_out, size_t(d) * sizeof(float)) != cudaSuccess) return GAR_ERR_CUDA;
        st->stage_out_elems = size_t(d);
    }
    if (!st->copy_stream) {
        if (cudaStreamCreateWithFlags(&st->copy_stream, cudaStreamNonBlocking) != cudaSuccess) return GAR_ERR_CUDA;
        if (cudaStreamCreateWithFlags(&st->compute_stream, cudaStreamNonBlocking) != cudaSuccess) return GAR_ERR_CUDA;
        if (cudaEventCreateWithFlags(&st->computed, cudaEventDisableTiming) != cudaSuccess) return GAR_ERR_CUDA;
    }
    // One bulk 2-D copy (row pitch d on both sides), then the device path; the
    // result goes back on the same stream.
    cudaStream_t s = st->compute_stream;
    if (cudaMemcpyAsync(st->stage_grads, grads, need * sizeof(float), cudaMemcpyHostToDevice, s) != cudaSuccess)
        return GAR_ERR_CUDA;
    Workspace ws{st->workspace};
    const int theta = default_theta(rule, n, f);
    rc = enqueue(rule, st->stage_grads, n, f, d, d, st->stage_out, 0, theta, 0, ws, nullptr, nullptr, st->sm_count, s);
    if (rc != GAR_OK) return rc;
    if (cudaMemcpyAsync(out, st->stage_out, size_t(d) * sizeof(float), cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return GAR_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return GAR_ERR_CUDA;
    return GAR_OK;
}

void gar_shutdown(void) {
    std::lock_guard<std::mutex> lock(g_mutex);
    int cur = 0;
    cudaGetDevice(&cur);
    for (int dev = 0; dev < kMaxDevices; ++dev) {
        DeviceState& st = g_dev[dev];
        if (!st.known) continue;
        cudaSetDevice(dev);
        cudaDeviceSynchronize();
        if (st.workspace) cudaFree(st.workspace);
        if (st.stage_grads) cudaFree(st.stage_grads);
        if (st.stage_out) cudaFree(st.stage_out);
        if (st.copy_stream) cudaStreamDestroy(st.copy_stream);
        if (st.compute_stream) cudaStreamDestroy(st.compute_stream);
        if (st.computed) cudaEventDestroy(st.computed);
        st = DeviceState{};
    }
    cudaSetDevice(cur);
}

}  // extern "C"
