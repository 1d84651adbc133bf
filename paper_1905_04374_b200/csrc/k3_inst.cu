// One instantiation of the coordinate kernel per compiled slot count K3_P
// (this file is compiled once for every entry of K3_P_LIST in k3_dispatch.cu;
// K3_EXACT = 1 when the kernel is only used with theta == K3_P).
#include "k3_bulk.cuh"

#if !defined(K3_P) || !defined(K3_EXACT)
#error "compile with -DK3_P=<slot count> -DK3_EXACT=<0|1>"
#endif

namespace gar {

// Threads per CTA and dynamic shared memory of the pre-aggregating kernel: every
// thread owns (loose_cap + GAR_MAX_SAVED) columns of V floats; aim at >= 2 CTAs per SM.
static inline void preagg_shape(int loose_cap, int V, int* threads, size_t* smem) {
    const size_t per_thread = size_t(loose_cap + GAR_MAX_SAVED) * V * sizeof(float);
    const size_t budget = 100 * 1024;
    int t = int(budget / per_thread) / 32 * 32;
    if (t > K3_THREADS) t = K3_THREADS;
    if (t < 32) t = 32;
    *threads = t;
    *smem = per_thread * t;
}

// Coordinates per thread of the staged kernel for this slot count (registers: 2 K3_P V values);
// measured on B200: 4 up to 12 slots with pre-aggregation (8 without), 2 up to 32, else 1.
template <bool PREAGG> struct BulkV { static constexpr int V = K3_P <= (PREAGG ? 12 : 8) ? 4 : (K3_P <= 32 ? 2 : 1); };

// Shared memory the staged kernel needs for one stage in the worst case (every gradient staged,
// a correction in every slot, theta * n additions in the plan).
static inline size_t bulk_pool_min(int n, int theta, int row_bytes) {
    return size_t((theta * n + 15) & ~15) + size_t(theta + 1) * row_bytes + size_t(n) * row_bytes;
}
constexpr size_t kBulkPerSm = 225 * 1024, kBulkPerCta = 3584;   // usable per SM; static shared memory + the system's share per CTA

template <bool PREAGG>
static int bulk_ctas(int n, int theta) {
    using S = KBShape<BulkV<PREAGG>::V>;
    int ctas = int(kBulkPerSm / (bulk_pool_min(n, theta, S::ROW_BYTES) + kBulkPerCta));
    const int by_threads = 2048 / S::THREADS;
    return ctas < by_threads ? ctas : by_threads;
}

// Full tiles [0, *covered) through the staged kernel, `ctas` CTAs per SM.
template <int P, bool PREAGG, bool H16>
static cudaError_t run_bulk(const float* g, int n, int64_t d, int64_t ld, gar_selection_t* sel, int theta,
                            int ctas, const K3Out& out, int sm_count, cudaStream_t stream, int64_t* covered, int dtype) {
    constexpr bool EXACT = (K3_EXACT != 0);
    constexpr int V = BulkV<PREAGG>::V;
    using S = KBShape<V>;
    *covered = 0;
    const int64_t ntiles = d / S::TC;
    if (ntiles == 0) return cudaSuccess;
    const size_t pool_min = bulk_pool_min(n, theta, S::ROW_BYTES);
    size_t pool = (kBulkPerSm / size_t(ctas) - kBulkPerCta) & ~size_t(127);
    const size_t pool_max = pool_min + size_t(KB_MAX_STAGES - 1) * n * S::ROW_BYTES;
    if (pool > pool_max) pool = pool_max;
    if (pool < pool_min) return cudaErrorInvalidValue;
    static size_t configured[64] = {0};
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= 64 || configured[dev] < pool) {
        err = cudaFuncSetAttribute(k3_bulk<P, EXACT, PREAGG, V, H16>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(pool));
        if (err != cudaSuccess) return err;
        err = cudaFuncSetAttribute(k3_bulk<P, EXACT, PREAGG, V, H16>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                   cudaSharedmemCarveoutMaxShared);
        if (err != cudaSuccess) return err;
        if (dev >= 0 && dev < 64) configured[dev] = pool;
    }
    int64_t grid = int64_t(sm_count) * ctas;
    if (grid > ntiles) grid = ntiles;
    k3_bulk<P, EXACT, PREAGG, V, H16><<<unsigned(grid), S::THREADS, pool, stream>>>(g, n, theta, ntiles, ld, sel, out, int(pool), dtype);
    *covered = ntiles * S::TC;
    return cudaGetLastError();
}

// Coordinates [t0, d): t0 is a multiple of 4.
template <int P, bool PREAGG, int V>
static cudaError_t run(const float* g, int n, int theta, int64_t t0, int64_t d, int64_t ld, gar_selection_t* sel, const K3Out& out,
                       int sm_count, cudaStream_t stream, int dtype) {
    constexpr bool EXACT = (K3_EXACT != 0);
    int threads = K3_THREADS, threads1 = K3_THREADS;
    size_t smem = 0, smem1 = 0;
    const int loose_cap = n < K3_LOOSE_CAP ? n : K3_LOOSE_CAP;
    if (PREAGG) {
        preagg_shape(loose_cap, V, &threads, &smem);
        preagg_shape(loose_cap, 1, &threads1, &smem1);
        static bool configured[64] = {false};      // per device, for this instantiation
        int dev = 0;
        cudaError_t err = cudaGetDevice(&dev);
        if (err != cudaSuccess) return err;
        if (!(dev >= 0 && dev < 64 && configured[dev])) {
            err = cudaFuncSetAttribute(k3_coordinate<P, EXACT, PREAGG, V>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
            if (err != cudaSuccess) return err;
            err = cudaFuncSetAttribute(k3_coordinate<P, EXACT, PREAGG, 1>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
            if (err != cudaSuccess) return err;
            err = cudaFuncSetAttribute(k3_coordinate<P, EXACT, PREAGG, V>,
                                       cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
            if (err != cudaSuccess) return err;
            if (dev >= 0 && dev < 64) configured[dev] = true;
        }
    }
    const int64_t d_vec = d - (d - t0) % V;
    if (d_vec > t0) {
        const int64_t nvec = (d_vec - t0) / V;
        int64_t blocks = (nvec + threads - 1) / threads;
        const int64_t cap = int64_t(sm_count) * 8;
        if (blocks > cap) blocks = cap;
        k3_coordinate<P, EXACT, PREAGG, V><<<unsigned(blocks), threads, smem, stream>>>(g, n, theta, t0, d_vec, ld, sel, out,
                                                                                         loose_cap, dtype);
    }
    if (d_vec < d) {   // ragged tail (only when ld > d): scalar kernel on the last d % V coordinates
        k3_coordinate<P, EXACT, PREAGG, 1><<<1, threads1, smem1, stream>>>(g, n, theta, d_vec, d, ld, sel, out, loose_cap, dtype);
    }
    return cudaGetLastError();
}

template <>
cudaError_t launch_k3_p<K3_P>(const float* g, int n, int64_t d, int64_t ld, gar_selection_t* sel, int theta, int preagg,
                              int vec, int bulk_ctas, const K3Out& out, int sm_count, cudaStream_t stream, int dtype) {
    int64_t t0 = 0;
    if (bulk_ctas > 0) {                         // whole tiles staged through shared memory, the rest below
        // 16-bit gradients: the staged kernel is compiled for the pre-aggregating rules only
        const cudaError_t err =
            dtype != GAR_F32 ? run_bulk<K3_P, true, true>(g, n, d, ld, sel, theta, bulk_ctas, out, sm_count, stream, &t0, dtype)
            : preagg         ? run_bulk<K3_P, true, false>(g, n, d, ld, sel, theta, bulk_ctas, out, sm_count, stream, &t0, dtype)
                             : run_bulk<K3_P, false, false>(g, n, d, ld, sel, theta, bulk_ctas, out, sm_count, stream, &t0, dtype);
        if (err != cudaSuccess) return err;
        if (t0 == d) return cudaSuccess;
    }
    // 4-wide vectors are only compiled for small slot counts (register budget)
    constexpr bool kWide = (K3_P <= 8);
    if (vec == 4 && !kWide) vec = 2;
    if (preagg) {
        if constexpr (kWide) if (vec == 4) return run<K3_P, true, 4>(g, n, theta, t0, d, ld, sel, out, sm_count, stream, dtype);
        if (vec == 2) return run<K3_P, true, 2>(g, n, theta, t0, d, ld, sel, out, sm_count, stream, dtype);
        return run<K3_P, true, 1>(g, n, theta, t0, d, ld, sel, out, sm_count, stream, dtype);
    }
    if constexpr (kWide) if (vec == 4) return run<K3_P, false, 4>(g, n, theta, t0, d, ld, sel, out, sm_count, stream, dtype);
    if (vec == 2) return run<K3_P, false, 2>(g, n, theta, t0, d, ld, sel, out, sm_count, stream, dtype);
    return run<K3_P, false, 1>(g, n, theta, t0, d, ld, sel, out, sm_count, stream, dtype);
}

// A batch of tensors through the register kernel, V coordinates per thread (every tensor's d, row
// stride and addresses allow V-wide accesses): one CTA per entry of cta_desc.
template <int P, bool PREAGG, int V>
static cudaError_t run_multi(const MultiDesc* desc, const int* cta_desc, int total_ctas, int n, int theta, gar_selection_t* sel,
                             int sel_stride, float lr, float mu, int dtype, cudaStream_t stream) {
    constexpr bool EXACT = (K3_EXACT != 0);
    int threads = K3_THREADS;
    size_t smem = 0;
    const int loose_cap = n < K3_LOOSE_CAP ? n : K3_LOOSE_CAP;
    if (PREAGG) {
        preagg_shape(loose_cap, V, &threads, &smem);
        static bool configured[64] = {false};      // per device, for this instantiation
        int dev = 0;
        cudaError_t err = cudaGetDevice(&dev);
        if (err != cudaSuccess) return err;
        if (!(dev >= 0 && dev < 64 && configured[dev])) {
            err = cudaFuncSetAttribute(k3_coordinate_multi<P, EXACT, PREAGG, V>, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
            if (err != cudaSuccess) return err;
            err = cudaFuncSetAttribute(k3_coordinate_multi<P, EXACT, PREAGG, V>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                       cudaSharedmemCarveoutMaxShared);
            if (err != cudaSuccess) return err;
            if (dev >= 0 && dev < 64) configured[dev] = true;
        }
    }
    k3_coordinate_multi<P, EXACT, PREAGG, V><<<unsigned(total_ctas), threads, smem, stream>>>(desc, cta_desc, n, theta, sel, sel_stride,
                                                                                              loose_cap, lr, mu, dtype);
    return cudaGetLastError();
}

// 4-wide vectors are only compiled for small slot counts (register budget)
static inline int multi_vec(int vec) { return (vec == 4 && K3_P > 8) ? 2 : vec; }

template <>
cudaError_t launch_k3_multi_p<K3_P>(const MultiDesc* desc, const int* cta_desc, int total_ctas, int n, int theta, int preagg,
                                    int vec, gar_selection_t* sel, int sel_stride, float lr, float mu, int dtype, cudaStream_t stream) {
    constexpr bool kWide = (K3_P <= 8);
    vec = multi_vec(vec);
    if (preagg) {
        if constexpr (kWide) if (vec == 4) return run_multi<K3_P, true, 4>(desc, cta_desc, total_ctas, n, theta, sel, sel_stride, lr, mu, dtype, stream);
        if (vec == 2) return run_multi<K3_P, true, 2>(desc, cta_desc, total_ctas, n, theta, sel, sel_stride, lr, mu, dtype, stream);
        return run_multi<K3_P, true, 1>(desc, cta_desc, total_ctas, n, theta, sel, sel_stride, lr, mu, dtype, stream);
    }
    if constexpr (kWide) if (vec == 4) return run_multi<K3_P, false, 4>(desc, cta_desc, total_ctas, n, theta, sel, sel_stride, lr, mu, dtype, stream);
    if (vec == 2) return run_multi<K3_P, false, 2>(desc, cta_desc, total_ctas, n, theta, sel, sel_stride, lr, mu, dtype, stream);
    return run_multi<K3_P, false, 1>(desc, cta_desc, total_ctas, n, theta, sel, sel_stride, lr, mu, dtype, stream);
}

// Threads per CTA of that launch.
template <>
int k3_multi_threads<K3_P>(int n, int preagg, int vec) {
    int threads = K3_THREADS;
    size_t smem = 0;
    if (preagg) preagg_shape(n < K3_LOOSE_CAP ? n : K3_LOOSE_CAP, multi_vec(vec), &threads, &smem);
    return threads;
}

// CTAs per SM the staged kernel would get for n gradients and theta slots (0: it cannot run).
template <>
int bulk_ctas_for<K3_P>(int n, int theta, int preagg) {
    return preagg ? bulk_ctas<true>(n, theta) : bulk_ctas<false>(n, theta);
}

}  // namespace gar
