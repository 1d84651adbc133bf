// One instantiation of the coordinate kernel per compiled slot count K3_P
// (this file is compiled once for every value in K3_P_LIST of k3_dispatch.cu).
#include "k3_coordinate.cuh"

#ifndef K3_P
#error "compile with -DK3_P=<slot count>"
#endif

namespace gar {

template <int P, bool PREAGG, int V>
static cudaError_t run(const float* g, int64_t d, int64_t ld, const gar_selection_t* sel, float* out,
                       int sm_count, cudaStream_t stream) {
    const int64_t d_vec = d - d % V;
    if (d_vec > 0) {
        const int64_t nvec = d_vec / V;
        int64_t blocks = (nvec + K3_THREADS - 1) / K3_THREADS;
        const int64_t cap = int64_t(sm_count) * 16;
        if (blocks > cap) blocks = cap;
        k3_coordinate<P, PREAGG, V><<<unsigned(blocks), K3_THREADS, 0, stream>>>(g, 0, d_vec, ld, sel, out);
    }
    if (d_vec < d) {   // ragged tail (only when ld > d): scalar kernel on the last d % V coordinates
        k3_coordinate<P, PREAGG, 1><<<1, K3_THREADS, 0, stream>>>(g, d_vec, d, ld, sel, out);
    }
    return cudaGetLastError();
}

template <>
cudaError_t launch_k3_p<K3_P>(const float* g, int64_t d, int64_t ld, const gar_selection_t* sel, int preagg,
                              int vec, float* out, int sm_count, cudaStream_t stream) {
    // 4-wide vectors are only compiled for small slot counts (register budget)
    constexpr bool kWide = (K3_P <= 8);
    if (vec == 4 && !kWide) vec = 2;
    if (preagg) {
        if constexpr (kWide) if (vec == 4) return run<K3_P, true, 4>(g, d, ld, sel, out, sm_count, stream);
        if (vec == 2) return run<K3_P, true, 2>(g, d, ld, sel, out, sm_count, stream);
        return run<K3_P, true, 1>(g, d, ld, sel, out, sm_count, stream);
    }
    if constexpr (kWide) if (vec == 4) return run<K3_P, false, 4>(g, d, ld, sel, out, sm_count, stream);
    if (vec == 2) return run<K3_P, false, 2>(g, d, ld, sel, out, sm_count, stream);
    return run<K3_P, false, 1>(g, d, ld, sel, out, sm_count, stream);
}

}  // namespace gar
