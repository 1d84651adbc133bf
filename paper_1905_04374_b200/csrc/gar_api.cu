// C ABI of libgar: argument validation, workspace handling and the enqueue of
// the three kernels (distances -> selection -> coordinate phase).
#include <algorithm>
#include <cstdio>
#include <mutex>
#include <vector>

#include "gar_internal.cuh"
#include "mbar.cuh"

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
    cudaStream_t host_stream = nullptr;   // gar_aggregate_host: copies and kernels, in order
};

DeviceState g_dev[kMaxDevices];
std::mutex  g_mutex;

// The CUDA error behind this thread's latest GAR_ERR_CUDA (gar_last_cuda_error).
thread_local cudaError_t t_last_cuda_error = cudaSuccess;
using gar::cuda_status;

}  // namespace

int gar::cuda_status(cudaError_t err) {
    if (err == cudaSuccess) return GAR_OK;
    t_last_cuda_error = err;
    return GAR_ERR_CUDA;
}

namespace {

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
    if (int rc_ = cuda_status(cudaGetDevice(&dev))) return rc_;
    if (dev < 0 || dev >= kMaxDevices) return GAR_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceState& st = g_dev[dev];
    if (!st.known) {
        if (int rc_ = cuda_status(cudaDeviceGetAttribute(&st.sm_count, cudaDevAttrMultiProcessorCount, dev))) return rc_;
        st.known = true;
    }
    if (need_workspace && !st.workspace) {
        if (int rc_ = cuda_status(cudaMalloc(&st.workspace, gar::kWorkspaceBytes))) return rc_;
        // the control block must read zero before the first kernel of ANY stream touches it (a
        // memset on the legacy stream is not ordered before work on a non-blocking stream)
        cudaError_t err = cudaMemset(st.workspace, 0, gar::kCtrlBytes);
        if (err == cudaSuccess) err = cudaDeviceSynchronize();
        if (err != cudaSuccess) {
            cudaFree(st.workspace);
            st.workspace = nullptr;
            return cuda_status(err);
        }
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
int enqueue(int rule, const float* grads, int n, int f, int64_t d, int64_t ld, const gar::K3Out& out, int m, int theta,
            int median_of_agr, int even_median, int distance_mode, const Workspace& ws, double* dist_out,
            gar_selection_t* sel_out, int sm_count, cudaStream_t stream, int dtype = GAR_F32) {
    const int beta = beta_for(rule, theta, f);
    double* dist = dist_out ? dist_out : ws.dist();
    gar_selection_t* sel = sel_out ? sel_out : ws.selection();
    cudaError_t err;
    const bool needs_dist = !(rule == GAR_AVERAGE || rule == GAR_MEDIAN);
    if (needs_dist) {
        err = dtype == GAR_F32 ? gar::launch_distances(grads, n, d, ld, dist, ws, sm_count, distance_mode, stream)
                               : gar::launch_distances_16(grads, dtype, n, d, ld, dist, ws, sm_count, stream);
        if (err != cudaSuccess) return cuda_status(err);
    }
    err = gar::launch_select(rule, dist, n, f, m, theta, beta, median_of_agr, even_median, sel, stream);
    if (err != cudaSuccess) return cuda_status(err);
    const int preagg = (rule == GAR_MULTI_BULYAN || rule == GAR_MULTI_KRUM || rule == GAR_AVERAGE) ? 1 : 0;
    err = gar::launch_coordinate(grads, n, d, ld, sel, theta, preagg, out, sm_count, stream, dtype);
    if (err != cudaSuccess) return cuda_status(err);
    return GAR_OK;
}

bool even_median_ok(int v) { return v == GAR_EVEN_MEDIAN_LOWER || v == GAR_EVEN_MEDIAN_MEAN; }
bool distance_mode_ok(int v) { return v == GAR_DISTANCES_AUTO || v == GAR_DISTANCES_DIFFERENCE; }

// One warp, a barrier that nothing arrives on, a bounded wait: it must give up.
__global__ void selftest_wait_kernel(unsigned limit, long long* result) {
    __shared__ unsigned long long bar;
    __shared__ int error_flag;
    if (threadIdx.x == 0) {
        gar::kb_init(&bar, 1u);
        error_flag = 0;
        gar::kb_fence_init();
    }
    __syncwarp();
    unsigned long long t0, t1;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    const bool ok = gar::kb_wait_warp(gar::kb_smem_u32(&bar), 0u, &error_flag, 4u, limit);
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
    if (threadIdx.x == 0) {
        result[0] = (!ok && error_flag) ? GAR_ERR_TIMEOUT : GAR_OK;
        result[1] = static_cast<long long>(t1 - t0);
    }
}

// dist = parts[0] + parts[1] + ... in that order (every GPU of a sharded aggregation runs this on
// the same gathered data and gets the same bits).
__global__ void reduce_partials_kernel(const double* __restrict__ parts, int count, int nn, double* __restrict__ dist) {
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= nn) return;
    double s = parts[idx];
    for (int r = 1; r < count; ++r) s += parts[size_t(r) * nn + idx];
    dist[idx] = s;
}

// ---- gar_aggregate_multi: workspace layout and the split of the work over CTAs
// CTAs beyond one per tensor that a batched launch may spend, shared out by length: upper bounds
// (they size the workspace); a call spends about one wave of resident CTAs, by the SM count.
constexpr int kMultiK1Budget = 1024, kMultiK3Budget = 2048;

struct MultiLayout {
    size_t tickets, table, dist, sel, partials, total;     // byte offsets; `table` = the host-built arrays
    size_t table_bytes;
    // inside the table
    size_t desc1, desc3, cta1, cta3;
};

MultiLayout multi_layout(int n, int count) {
    MultiLayout L{};
    size_t off = 0;
    L.tickets = off;  off += gar::align256(size_t(count + 1) * sizeof(unsigned int));   // + the staged kernel's error word
    L.table = off;
    size_t t = 0;
    L.desc1 = t;  t += gar::align256(size_t(count) * sizeof(gar::MultiDesc));
    L.desc3 = t;  t += gar::align256(size_t(count) * sizeof(gar::MultiDesc));
    L.cta1 = t;   t += gar::align256(size_t(count + kMultiK1Budget) * sizeof(int));
    L.cta3 = t;   t += gar::align256(size_t(count + kMultiK3Budget) * sizeof(int));
    L.table_bytes = t;
    off += t;
    L.dist = off;     off += gar::align256(size_t(count + 1) * n * n * sizeof(double));
    L.sel = off;      off += gar::align256(size_t(count) * sizeof(gar_selection_t));
    L.partials = off; off += size_t(count + kMultiK1Budget) * gar::kPairSlots * sizeof(double);
    L.total = off;
    return L;
}

// CTAs of one tensor: one, plus its share (by length) of the budget, at most `useful`.
int multi_ctas(int64_t d, double total_d, int budget, int64_t useful) {
    int64_t c = 1 + int64_t(double(budget) * double(d) / total_d);
    if (c > useful) c = useful;
    return c < 1 ? 1 : int(c);
}

}  // namespace

namespace gar {
cudaError_t launch_selftest_wait(unsigned limit, long long* result, cudaStream_t stream) {
    selftest_wait_kernel<<<1, 32, 0, stream>>>(limit, result);
    return cudaGetLastError();
}
}  // namespace gar

extern "C" {

int gar_version(void) { return GAR_VERSION; }

int gar_last_cuda_error(void) { return int(t_last_cuda_error); }
const char* gar_last_cuda_error_name(void) { return cudaGetErrorName(t_last_cuda_error); }

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
    if (!p->grads || (!p->out && !p->sgd_params)) return GAR_ERR_INVALID_ARG;
    if (p->sgd_momentum_buf && !p->sgd_params) return GAR_ERR_INVALID_ARG;
    const int64_t ld = p->ld ? p->ld : p->d;
    if (ld < p->d) return GAR_ERR_INVALID_ARG;
    if (p->grads_dtype != GAR_F32 && p->grads_dtype != GAR_BF16 && p->grads_dtype != GAR_F16) return GAR_ERR_INVALID_ARG;
    {
        const size_t esize = p->grads_dtype == GAR_F32 ? sizeof(float) : 2;
        const size_t gbytes = (size_t(p->n - 1) * ld + p->d) * esize, vbytes = size_t(p->d) * sizeof(float);
        const float* vecs[3] = {p->out, p->sgd_params, p->sgd_momentum_buf};
        for (int a = 0; a < 3; ++a) {
            if (!vecs[a]) continue;
            if (overlaps(p->grads, gbytes, vecs[a], vbytes)) return GAR_ERR_INVALID_ARG;
            for (int b = a + 1; b < 3; ++b)
                if (vecs[b] && overlaps(vecs[a], vbytes, vecs[b], vbytes)) return GAR_ERR_INVALID_ARG;
        }
    }
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
    if (!even_median_ok(p->even_median) || !distance_mode_ok(p->distance_mode)) return GAR_ERR_INVALID_ARG;
    DeviceState* st = nullptr;
    Workspace ws{};
    rc = resolve_workspace(p->workspace, p->workspace_bytes, &st, &ws);
    if (rc != GAR_OK) return rc;
    const gar::K3Out out{p->out, p->sgd_params, p->sgd_momentum_buf, p->sgd_lr, p->sgd_momentum};
    return enqueue(p->rule, p->grads, p->n, p->f, p->d, ld, out, m, theta, p->median_of_agr, p->even_median,
                   p->distance_mode, ws, p->dist_out, p->selection_out, st->sm_count,
                   static_cast<cudaStream_t>(p->stream), p->grads_dtype);
}

int gar_aggregate(int rule, const float* grads, int n, int f, int64_t d, float* out, void* stream) {
    gar_params_t p{};
    p.rule = rule; p.n = n; p.f = f; p.d = d; p.ld = d;
    p.grads = grads; p.out = out; p.stream = stream;
    return gar_aggregate_ex(&p);
}

int gar_pairwise_distances(const float* grads, int n, int64_t d, int64_t ld, double* dist, void* workspace,
                           size_t workspace_bytes, void* stream) {
    return gar_pairwise_distances_mode(grads, n, d, ld, dist, workspace, workspace_bytes, GAR_DISTANCES_AUTO, stream);
}

int gar_pairwise_distances_mode(const float* grads, int n, int64_t d, int64_t ld, double* dist, void* workspace,
                                size_t workspace_bytes, int distance_mode, void* stream) {
    if (!grads || !dist || n < 1 || d < 1 || !distance_mode_ok(distance_mode)) return GAR_ERR_INVALID_ARG;
    if (n > GAR_MAX_N) return GAR_ERR_UNSUPPORTED;
    if (ld == 0) ld = d;
    if (ld < d) return GAR_ERR_INVALID_ARG;
    DeviceState* st = nullptr;
    Workspace ws{};
    int rc = resolve_workspace(workspace, workspace_bytes, &st, &ws);
    if (rc != GAR_OK) return rc;
    cudaError_t err = gar::launch_distances(grads, n, d, ld, dist, ws, st->sm_count, distance_mode,
                                            static_cast<cudaStream_t>(stream));
    return cuda_status(err);
}

int gar_select(int rule, const double* dist, int n, int f, int m, int theta, int median_of_agr, int even_median,
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
    if (!even_median_ok(even_median)) return GAR_ERR_INVALID_ARG;
    cudaError_t err = gar::launch_select(rule, dist, n, f, m, th, beta_for(rule, th, f), median_of_agr, even_median, sel,
                                         static_cast<cudaStream_t>(stream));
    return cuda_status(err);
}

int gar_schedule_from_tables(gar_selection_t* sel, void* stream) {
    if (!sel) return GAR_ERR_INVALID_ARG;
    cudaError_t err = gar::launch_schedule_only(sel, static_cast<cudaStream_t>(stream));
    return cuda_status(err);
}

int gar_coordinate_phase(const float* grads, int n, int64_t d, int64_t ld, gar_selection_t* sel, int theta,
                         int preagg, float* out, void* stream) {
    if (!grads || !sel || !out || n < 1 || d < 1 || theta < 1 || theta > GAR_MAX_N) return GAR_ERR_INVALID_ARG;
    if (n > GAR_MAX_N) return GAR_ERR_UNSUPPORTED;
    if (ld == 0) ld = d;
    if (ld < d) return GAR_ERR_INVALID_ARG;
    DeviceState* st = nullptr;
    int rc = device_state(&st, false);
    if (rc != GAR_OK) return rc;
    const gar::K3Out o{out, nullptr, nullptr, 0.0f, 0.0f};
    cudaError_t err = gar::launch_coordinate(grads, n, d, ld, sel, theta, preagg ? 1 : 0, o, st->sm_count,
                                             static_cast<cudaStream_t>(stream));
    return cuda_status(err);
}

int gar_reduce_partials(const double* parts, int count, int n, double* dist, void* stream) {
    if (!parts || !dist || count < 1 || count > 1024 || n < 1) return GAR_ERR_INVALID_ARG;
    if (n > GAR_MAX_N) return GAR_ERR_UNSUPPORTED;
    const int nn = n * n;
    reduce_partials_kernel<<<(nn + 255) / 256, 256, 0, static_cast<cudaStream_t>(stream)>>>(parts, count, nn, dist);
    return cuda_status(cudaGetLastError());
}

size_t gar_multi_workspace_bytes(int rule, int n, int f, int count) {
    if (basic_checks(rule, n, f, 1) != GAR_OK || count < 1) return 0;
    return multi_layout(n, count).total;
}

int gar_aggregate_multi(const gar_multi_params_t* p) {
    if (!p) return GAR_ERR_INVALID_ARG;
    int rc = basic_checks(p->rule, p->n, p->f, 1);
    if (rc != GAR_OK) return rc;
    if (p->count < 1 || !p->tensors || (p->joint != 0 && p->joint != 1) || !even_median_ok(p->even_median))
        return GAR_ERR_INVALID_ARG;
    if (p->grads_dtype != GAR_F32 && p->grads_dtype != GAR_BF16 && p->grads_dtype != GAR_F16) return GAR_ERR_INVALID_ARG;
    const int dtype = p->grads_dtype;
    const size_t esize = dtype == GAR_F32 ? sizeof(float) : 2;
    const int n = p->n, count = p->count;
    for (int t = 0; t < count; ++t) {
        const gar_tensor_t& x = p->tensors[t];
        const int64_t ld = x.ld ? x.ld : x.d;
        if (!x.grads || (!x.out && !x.sgd_params) || x.d < 1 || ld < x.d) return GAR_ERR_INVALID_ARG;
        if (x.sgd_momentum_buf && !x.sgd_params) return GAR_ERR_INVALID_ARG;
    }
    {
        // no output may overlap a gradient block or another output, of any tensor: sweep over the
        // address ranges in order of their start
        struct Range { uintptr_t begin, end; bool is_out; };
        std::vector<Range> ranges;
        ranges.reserve(4 * size_t(count));
        for (int t = 0; t < count; ++t) {
            const gar_tensor_t& x = p->tensors[t];
            const int64_t ld = x.ld ? x.ld : x.d;
            const uintptr_t g0 = reinterpret_cast<uintptr_t>(x.grads);
            ranges.push_back({g0, g0 + (size_t(n - 1) * ld + x.d) * esize, false});
            const float* outs[3] = {x.out, x.sgd_params, x.sgd_momentum_buf};
            for (const float* o : outs) {
                if (!o) continue;
                const uintptr_t o0 = reinterpret_cast<uintptr_t>(o);
                ranges.push_back({o0, o0 + size_t(x.d) * sizeof(float), true});
            }
        }
        std::sort(ranges.begin(), ranges.end(), [](const Range& a, const Range& b) { return a.begin < b.begin; });
        uintptr_t end_any = 0, end_out = 0;
        for (const Range& r : ranges) {
            if (r.begin < (r.is_out ? end_any : end_out)) return GAR_ERR_INVALID_ARG;
            if (r.end > end_any) end_any = r.end;
            if (r.is_out && r.end > end_out) end_out = r.end;
        }
    }
    const MultiLayout L = multi_layout(n, count);
    if (!p->workspace || reinterpret_cast<uintptr_t>(p->workspace) % 256 != 0 || p->workspace_bytes < L.total)
        return GAR_ERR_WORKSPACE;
    DeviceState* st = nullptr;
    rc = device_state(&st, false);
    if (rc != GAR_OK) return rc;
    char* const ws = static_cast<char*>(p->workspace);
    cudaStream_t stream = static_cast<cudaStream_t>(p->stream);
    const int rule = p->rule, f = p->f;
    const int theta = default_theta(rule, n, f), beta = beta_for(rule, theta, f);
    const int preagg = (rule == GAR_MULTI_BULYAN || rule == GAR_MULTI_KRUM || rule == GAR_AVERAGE) ? 1 : 0;
    const bool needs_dist = !(rule == GAR_AVERAGE || rule == GAR_MEDIAN);

    // one wave: the ring kernel keeps three CTAs per SM resident, the tiled kernel two, the register kernel six
    const int k1_budget = std::min(kMultiK1Budget, ((n <= 16 && p->grads_dtype == GAR_F32) ? 3 : 2) * st->sm_count);
    const int k3_budget = std::min(kMultiK3Budget, 6 * st->sm_count);
    // ---- the host-built table: descriptors in launch order (wide-access tensors first) and the CTA lists
    std::vector<char> table(L.table_bytes, 0);
    gar::MultiDesc* desc1 = reinterpret_cast<gar::MultiDesc*>(table.data() + L.desc1);
    gar::MultiDesc* desc3 = reinterpret_cast<gar::MultiDesc*>(table.data() + L.desc3);
    int* cta1 = reinterpret_cast<int*>(table.data() + L.cta1);
    int* cta3 = reinterpret_cast<int*>(table.data() + L.cta3);
    auto fill = [&](gar::MultiDesc& m, int t) {
        const gar_tensor_t& x = p->tensors[t];
        m.grads = x.grads; m.out = x.out; m.x = x.sgd_params; m.v = x.sgd_momentum_buf; m.d = x.d; m.ld = x.ld ? x.ld : x.d; m.index = t; m.ctas = 1; m.cta_first = 0; m.pad = 0;
    };
    // distances: classes by the alignment of the rows, 16 / 8 / 4 bytes; up to 16 rows, long
    // tensors of the first class form a class of their own (the staged kernel, one CTA per SM)
    const int widths[3] = {4, 2, 1};
    const int k1_class[4] = {gar::kMultiStaged, 4, 2, 1};
    int first1[5] = {0, 0, 0, 0, 0}, ctas1[4] = {0, 0, 0, 0};
    {
        int pos = 0, cta_off = 0;
        for (int cls = 0; cls < 4; ++cls) {
            first1[cls] = pos;
            const int chunk = gar::distances_multi_chunk(n, k1_class[cls], dtype);
            auto class_of = [&](const gar_tensor_t& x) {
                const int64_t ld = x.ld ? x.ld : x.d;
                const uintptr_t addr = reinterpret_cast<uintptr_t>(x.grads);
                if (dtype != GAR_F32)     // 16-bit: the staged kernel (rows 16-byte aligned), else element by element
                    return (n <= 16 && addr % 16 == 0 && ld % 8 == 0 && x.d >= gar::kMultiStagedMinDim) ? 0 : 3;
                const int c = (addr % 16 == 0 && ld % 4 == 0) ? 1 : ((addr % 8 == 0 && ld % 2 == 0) ? 2 : 3);
                return (c == 1 && n <= 16 && x.d >= gar::kMultiStagedMinDim) ? 0 : c;
            };
            // the class's CTAs, the one per tensor included, stay within one wave of resident CTAs
            // (the staged kernel holds a whole SM); the rest of the wave is shared out by length
            int members = 0;
            double class_d = 0.0;
            for (int t = 0; t < count; ++t)
                if (class_of(p->tensors[t]) == cls) { ++members; class_d += double(p->tensors[t].d); }
            if (members == 0) continue;
            const int wave = cls == 0 ? st->sm_count : k1_budget;
            const int budget = wave > members ? wave - members : 0;
            int cta = 0;
            for (int t = 0; t < count; ++t) {
                const gar_tensor_t& x = p->tensors[t];
                if (class_of(x) != cls) continue;
                gar::MultiDesc& m = desc1[pos];
                fill(m, t);
                m.ctas = multi_ctas(x.d, class_d, budget, (x.d + chunk - 1) / chunk);
                m.cta_first = cta;
                for (int c = 0; c < m.ctas; ++c) cta1[cta_off + cta + c] = pos - first1[cls];
                cta += m.ctas;
                ++pos;
            }
            ctas1[cls] = cta;
            cta_off += cta;
        }
        first1[4] = pos;
    }
    // coordinate phase: classes by vector width 4, 2, 1
    int first3[4] = {0, 0, 0, 0}, ctas3[3] = {0, 0, 0};
    {
        int pos = 0, cta_off = 0;
        for (int cls = 0; cls < 3; ++cls) {
            first3[cls] = pos;
            const int threads = gar::coordinate_multi_threads(n, theta, preagg, widths[cls]);
            auto class_of = [&](const gar_tensor_t& x) {
                return gar::coordinate_multi_vec(x.grads, x.out, x.sgd_params, x.sgd_momentum_buf, x.d, x.ld ? x.ld : x.d, theta, preagg, dtype);
            };
            int members = 0;
            double class_d = 0.0;
            for (int t = 0; t < count; ++t)
                if (class_of(p->tensors[t]) == widths[cls]) { ++members; class_d += double(p->tensors[t].d); }
            if (members == 0) continue;
            const int budget = k3_budget > members ? k3_budget - members : 0;
            int cta = 0;
            for (int t = 0; t < count; ++t) {
                const gar_tensor_t& x = p->tensors[t];
                if (class_of(x) != widths[cls]) continue;
                gar::MultiDesc& m = desc3[pos];
                fill(m, t);
                const int64_t per_cta = int64_t(threads) * widths[cls];
                m.ctas = multi_ctas(x.d, class_d, budget, (x.d + per_cta - 1) / per_cta);
                m.cta_first = cta;
                for (int c = 0; c < m.ctas; ++c) cta3[cta_off + cta + c] = pos - first3[cls];
                cta += m.ctas;
                ++pos;
            }
            ctas3[cls] = cta;
            cta_off += cta;
        }
        first3[3] = pos;
    }
    if (int e = cuda_status(cudaMemcpyAsync(ws + L.table, table.data(), L.table_bytes, cudaMemcpyHostToDevice, stream))) return e;
    // the pageable source has been staged when the copy call returns; `table` may go out of scope

    const gar::MultiDesc* d_desc1 = reinterpret_cast<const gar::MultiDesc*>(ws + L.table + L.desc1);
    const gar::MultiDesc* d_desc3 = reinterpret_cast<const gar::MultiDesc*>(ws + L.table + L.desc3);
    const int* d_cta1 = reinterpret_cast<const int*>(ws + L.table + L.cta1);
    const int* d_cta3 = reinterpret_cast<const int*>(ws + L.table + L.cta3);
    double* ws_dist = reinterpret_cast<double*>(ws + L.dist);
    gar_selection_t* sel = p->selection_out ? p->selection_out : reinterpret_cast<gar_selection_t*>(ws + L.sel);
    // independent problems: the matrices go where the caller wants them; joint: the pieces stay in
    // the workspace and their sum goes there
    double* dist_each = (!p->joint && p->dist_out) ? p->dist_out : ws_dist;
    double* dist_joint = p->dist_out ? p->dist_out : ws_dist + size_t(count) * n * n;

    if (needs_dist) {
        if (int e = cuda_status(cudaMemsetAsync(ws + L.tickets, 0, size_t(count + 1) * sizeof(unsigned int), stream))) return e;
        double* partials = reinterpret_cast<double*>(ws + L.partials);
        unsigned int* tickets = reinterpret_cast<unsigned int*>(ws + L.tickets);
        int cta_off = 0;
        for (int cls = 0; cls < 4; ++cls) {
            if (ctas1[cls] == 0) continue;
            const cudaError_t err = gar::launch_distances_multi(d_desc1 + first1[cls], d_cta1 + cta_off, ctas1[cls], n, k1_class[cls],
                                                                dist_each, partials + size_t(cta_off) * gar::kPairSlots, tickets,
                                                                tickets + count, dtype, stream);
            if (err != cudaSuccess) return cuda_status(err);
            cta_off += ctas1[cls];
        }
        if (p->joint) {
            const int nn = n * n;
            reduce_partials_kernel<<<(nn + 255) / 256, 256, 0, stream>>>(dist_each, count, nn, dist_joint);
            if (int e = cuda_status(cudaGetLastError())) return e;
        }
    }
    {
        const cudaError_t err = gar::launch_select(rule, p->joint ? dist_joint : dist_each, n, f, 0, theta, beta, 0, p->even_median,
                                                   sel, stream, p->joint ? 1 : count);
        if (err != cudaSuccess) return cuda_status(err);
    }
    {
        int cta_off = 0;
        for (int cls = 0; cls < 3; ++cls) {
            if (ctas3[cls] == 0) continue;
            const cudaError_t err = gar::launch_coordinate_multi(d_desc3 + first3[cls], d_cta3 + cta_off, ctas3[cls], n, theta, preagg,
                                                                 widths[cls], sel, p->joint ? 0 : 1, p->sgd_lr, p->sgd_momentum, dtype, stream);
            if (err != cudaSuccess) return cuda_status(err);
            cta_off += ctas3[cls];
        }
    }
    return GAR_OK;
}

int gar_selftest_bounded_wait(unsigned int limit, long long* result, void* stream) {
    if (!result || limit < 1u || limit > 65536u) return GAR_ERR_INVALID_ARG;
    return cuda_status(gar::launch_selftest_wait(limit, result, static_cast<cudaStream_t>(stream)));
}

int gar_aggregate_host(int rule, const float* grads, int n, int f, int64_t d, float* out) {
    int rc = basic_checks(rule, n, f, d);
    if (rc != GAR_OK) return rc;
    if (!grads || !out) return GAR_ERR_INVALID_ARG;
    DeviceState* st = nullptr;
    rc = device_state(&st, true);
    if (rc != GAR_OK) return rc;
    // staging buffers and the stream (cached, grown on demand, under the lock; the call itself
    // uses them outside it: concurrent host calls on one device must be serialised by the caller)
    const size_t need = size_t(n) * size_t(d);
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        if (st->stage_grads_elems < need) {
            if (st->stage_grads) cudaFree(st->stage_grads);
            st->stage_grads = nullptr; st->stage_grads_elems = 0;
            if (int rc_ = cuda_status(cudaMalloc(&st->stage_grads, need * sizeof(float)))) return rc_;
            st->stage_grads_elems = need;
        }
        if (st->stage_out_elems < size_t(d)) {
            if (st->stage_out) cudaFree(st->stage_out);
            st->stage_out = nullptr; st->stage_out_elems = 0;
            if (int rc_ = cuda_status(cudaMalloc(&st->stage_out, size_t(d) * sizeof(float)))) return rc_;
            st->stage_out_elems = size_t(d);
        }
        if (!st->host_stream) {
            if (int rc_ = cuda_status(cudaStreamCreateWithFlags(&st->host_stream, cudaStreamNonBlocking))) return rc_;
        }
    }
    // rows in (one contiguous copy), the three kernels, the result and the selection's status out
    cudaStream_t s = st->host_stream;
    if (int rc_ = cuda_status(cudaMemcpyAsync(st->stage_grads, grads, need * sizeof(float), cudaMemcpyHostToDevice, s))) return rc_;
    Workspace ws{st->workspace};
    const int theta = default_theta(rule, n, f);
    const gar::K3Out stage_out{st->stage_out, nullptr, nullptr, 0.0f, 0.0f};
    rc = enqueue(rule, st->stage_grads, n, f, d, d, stage_out, 0, theta, 0, GAR_EVEN_MEDIAN_LOWER, GAR_DISTANCES_AUTO,
                 ws, nullptr, nullptr, st->sm_count, s);
    if (rc != GAR_OK) return rc;
    if (int rc_ = cuda_status(cudaMemcpyAsync(out, st->stage_out, size_t(d) * sizeof(float), cudaMemcpyDeviceToHost, s))) return rc_;
    int32_t status = GAR_OK;
    if (int rc_ = cuda_status(cudaMemcpyAsync(&status, &ws.selection()->status, sizeof(status), cudaMemcpyDeviceToHost, s))) return rc_;
    if (int rc_ = cuda_status(cudaStreamSynchronize(s))) return rc_;
    return status;
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
        if (st.host_stream) cudaStreamDestroy(st.host_stream);
        st = DeviceState{};
    }
    cudaSetDevice(cur);
}

}  // extern "C"
