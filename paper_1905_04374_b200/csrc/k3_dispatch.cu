// Chooses the compiled slot count and vector width of the coordinate kernel.
#include "gar_internal.cuh"

// Slot counts the coordinate kernel is compiled for (k3_inst.cu is built once
// per entry; keep the build script's list identical): every theta up to 32 has
// its own kernel with theta fixed at compile time; larger ones share padded kernels.
#define K3_P_LIST(X)                                                                                   \
    X(1) X(2) X(3) X(4) X(5) X(6) X(7) X(8) X(9) X(10) X(11) X(12) X(13) X(14) X(15) X(16) X(17) X(18) \
    X(19) X(20) X(21) X(22) X(23) X(24) X(25) X(26) X(27) X(28) X(29) X(30) X(31) X(32) X(36) X(40)    \
    X(44) X(48) X(52) X(56) X(60) X(64)

namespace gar {

template <int P>
cudaError_t launch_k3_p(const float* g, int n, int64_t d, int64_t ld, gar_selection_t* sel, int theta, int preagg,
                        int vec, int bulk_ctas, const K3Out& out, int sm_count, cudaStream_t stream, int dtype);
template <int P> int bulk_ctas_for(int n, int theta, int preagg);
template <int P>
cudaError_t launch_k3_multi_p(const MultiDesc* desc, const int* cta_desc, int total_ctas, int n, int theta, int preagg, int vec,
                              gar_selection_t* sel, int sel_stride, float lr, float mu, int dtype, cudaStream_t stream);
template <int P> int k3_multi_threads(int n, int preagg, int vec);
#define K3_DECL(P)                                                                                              \
    template <>                                                                                                 \
    cudaError_t launch_k3_p<P>(const float*, int, int64_t, int64_t, gar_selection_t*, int, int, int, int,       \
                               const K3Out&, int, cudaStream_t, int);                                                    \
    template <> int bulk_ctas_for<P>(int, int, int);                                                            \
    template <>                                                                                                 \
    cudaError_t launch_k3_multi_p<P>(const MultiDesc*, const int*, int, int, int, int, int, gar_selection_t*, int, float, float, \
                                     int, cudaStream_t); \
    template <> int k3_multi_threads<P>(int, int, int);
K3_P_LIST(K3_DECL)
#undef K3_DECL

cudaError_t launch_coordinate(const float* grads, int n, int64_t d, int64_t ld, gar_selection_t* sel,
                              int theta, int preagg, const K3Out& out, int sm_count, cudaStream_t stream, int dtype) {
    const uintptr_t o = reinterpret_cast<uintptr_t>(out.out) | reinterpret_cast<uintptr_t>(out.x) |
                        reinterpret_cast<uintptr_t>(out.v);
    const uintptr_t a = reinterpret_cast<uintptr_t>(grads) | o;
    int vec_max = 1;                                      // what the alignment allows
    if (dtype == GAR_F32) {
        if (a % 16 == 0 && ld % 4 == 0) vec_max = 4;
        else if (a % 8 == 0 && ld % 2 == 0) vec_max = 2;
    } else {                                              // V 16-bit elements per load, V floats per store
        const uintptr_t ga = reinterpret_cast<uintptr_t>(grads);
        if (ga % 8 == 0 && o % 16 == 0 && ld % 4 == 0) vec_max = 4;
        else if (ga % 4 == 0 && o % 8 == 0 && ld % 2 == 0) vec_max = 2;
    }
    // widest width that keeps the kernel's registers in check: large slot counts use narrower vectors
    int vec = vec_max;
    if (vec == 4 && theta > 8) vec = 2;
    if (vec == 2 && theta > (preagg ? 12 : 24)) vec = 1;
    // Staging through shared memory by bulk copies needs 16-byte aligned row segments.  With
    // pre-aggregation it is the faster kernel at every slot count; without (Bulyan, median, Krum:
    // the winners are all that is read) the register kernel with 2- or 4-wide loads keeps up with
    // memory and wins while the slot count is a compile-time constant, up to 32 slots.
    const int bulk_from = preagg ? 1 : 33;
    // (a few hundred thousand coordinates amortise its set-up: the plan, the barriers, the first tiles)
    // (16-bit gradients: staged for the pre-aggregating rules when the rows are 16-byte aligned,
    // else through the register kernel, which widens them as it loads)
    const bool rows16 = dtype != GAR_F32 && preagg && reinterpret_cast<uintptr_t>(grads) % 16 == 0 && ld % 8 == 0 && o % 16 == 0;
    const bool bulk = (dtype == GAR_F32 ? vec_max == 4 : rows16) && theta >= bulk_from && d >= 400000;
#define K3_TRY(P)                                                                                              \
    if (theta <= P) {                                                                                          \
        const int ctas = bulk ? bulk_ctas_for<P>(n, theta, preagg) : 0;                                        \
        return launch_k3_p<P>(grads, n, d, ld, sel, theta, preagg, vec, ctas, out, sm_count, stream, dtype);   \
    }
    K3_P_LIST(K3_TRY)
#undef K3_TRY
    return cudaErrorInvalidValue;
}

// Vector width of the register kernel for one tensor of a batch: what its addresses, row stride
// and length allow (the batched kernel has no ragged-tail pass, so d must be a multiple too),
// narrowed as launch_coordinate narrows it for large slot counts.
int coordinate_multi_vec(const void* grads, const void* out, const void* x, const void* v, int64_t d, int64_t ld, int theta,
                         int preagg, int dtype) {
    const uintptr_t g = reinterpret_cast<uintptr_t>(grads);
    const uintptr_t o = reinterpret_cast<uintptr_t>(out) | reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(v);
    int vec = 1;
    if (dtype == GAR_F32) {
        if ((g | o) % 16 == 0 && ld % 4 == 0 && d % 4 == 0) vec = 4;
        else if ((g | o) % 8 == 0 && ld % 2 == 0 && d % 2 == 0) vec = 2;
    } else {                                              // V 16-bit elements per load, V floats per store
        if (g % 8 == 0 && o % 16 == 0 && ld % 4 == 0 && d % 4 == 0) vec = 4;
        else if (g % 4 == 0 && o % 8 == 0 && ld % 2 == 0 && d % 2 == 0) vec = 2;
    }
    if (vec == 4 && theta > 8) vec = 2;
    if (vec == 2 && theta > (preagg ? 12 : 24)) vec = 1;
    return vec;
}

cudaError_t launch_coordinate_multi(const MultiDesc* desc, const int* cta_desc, int total_ctas, int n, int theta, int preagg,
                                    int vec, gar_selection_t* sel, int sel_stride, float lr, float mu, int dtype, cudaStream_t stream) {
#define K3_TRY(P) \
    if (theta <= P) return launch_k3_multi_p<P>(desc, cta_desc, total_ctas, n, theta, preagg, vec, sel, sel_stride, lr, mu, dtype, stream);
    K3_P_LIST(K3_TRY)
#undef K3_TRY
    return cudaErrorInvalidValue;
}

int coordinate_multi_threads(int n, int theta, int preagg, int vec) {
#define K3_TRY(P) \
    if (theta <= P) return k3_multi_threads<P>(n, preagg, vec);
    K3_P_LIST(K3_TRY)
#undef K3_TRY
    return 128;
}

}  // namespace gar
