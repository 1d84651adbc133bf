// Internal declarations shared by the translation units of libgar.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "gar.h"

namespace gar {

// ---- workspace layout (device) -------------------------------------------
// [0, 256)                control block, 32-bit words: [0] ticket counter of the distance kernel,
//                          [2] a bounded wait of a distance kernel gave up, [4] path of the last
//                          distance call (kPath*), [6] gate of the difference-form kernel that follows
//                          the tensor-core kernel (non-zero: recompute)
// [256, +partials)        per-CTA partial distance sums, fp64
// [.., +n*n doubles)      distance matrix
// [.., +sizeof(selection)) selection result / coordinate-phase schedule
constexpr int    kMaxCtasK1      = 592;                 // upper bound on the distance kernel's grid
constexpr int    kMaxTiles       = 36;                  // 8x8 row-block pairs at n = 64
constexpr int    kPairSlots      = kMaxTiles * 64;      // fp64 slots per CTA partial
constexpr size_t kCtrlBytes      = 256;
constexpr size_t kPartialBytes   = size_t(kMaxCtasK1) * kPairSlots * sizeof(double);
constexpr size_t kDistBytes      = size_t(GAR_MAX_N) * GAR_MAX_N * sizeof(double);

constexpr size_t align256(size_t x) { return (x + 255) & ~size_t(255); }

constexpr size_t kOffPartials  = kCtrlBytes;
constexpr size_t kOffDist      = kOffPartials + align256(kPartialBytes);
constexpr size_t kOffSelection = kOffDist + align256(kDistBytes);
constexpr size_t kWorkspaceBytes = kOffSelection + align256(sizeof(gar_selection_t));

struct Workspace {
    char* base;
    unsigned int*    ticket()    const { return reinterpret_cast<unsigned int*>(base); }
    unsigned int*    k1_error()  const { return reinterpret_cast<unsigned int*>(base) + 2; }   // a bounded device wait gave up
    unsigned int*    k1_path()   const { return reinterpret_cast<unsigned int*>(base) + 4; }
    unsigned int*    k1_gate()   const { return reinterpret_cast<unsigned int*>(base) + 6; }
    double*          partials()  const { return reinterpret_cast<double*>(base + kOffPartials); }
    double*          dist()      const { return reinterpret_cast<double*>(base + kOffDist); }
    gar_selection_t* selection() const { return reinterpret_cast<gar_selection_t*>(base + kOffSelection); }
};

constexpr unsigned kPathDifference = 0u, kPathGram = 1u, kPathGramRejected = 2u;

// Slots of a CTA's partial-sum block beyond the pair sums.
constexpr int kSlotRowExp    = 2100;    // .. +63: the tensor-core kernel's final quantisation exponent of each row
constexpr int kSlotNonfinite = 2300;    // 2300, 2301: masks of rows that hold Inf or NaN
constexpr int kSlotError     = 2302;    // a bounded wait gave up

// One tensor of a batched call (gar_aggregate_multi): the device copy of a gar_tensor_t, the
// tensor's place in the caller's array (it addresses the tensor's distance matrix, selection and
// ticket) and its share of the launch: CTAs cta_first .. cta_first + ctas - 1 of a one-dimensional
// grid, sized by the tensor's length.  A second array maps every CTA to its descriptor.
struct MultiDesc {
    const void* grads;
    float*      out;
    float*      x;          // fused SGD step: parameters and momentum buffer (may be null)
    float*      v;
    int64_t     d, ld;
    int         index;
    int         ctas, cta_first;
    int         pad;
};

// Where the coordinate kernel puts a coordinate's result: the aggregate itself (out, may be null
// when a step is fused) and/or an SGD step on x with optional momentum buffer v (Eq. 2).
struct K3Out {
    float* out;
    float* x;
    float* v;
    float  lr, mu;
};

// ---- 16-bit gradients ---------------------------------------------------------------------
// One 16-bit element (bfloat16 or binary16, by `dtype`) widened to fp32, exactly.
__device__ __forceinline__ float widen16(unsigned short raw, int dtype) {
    if (dtype == GAR_BF16) return __uint_as_float(static_cast<unsigned>(raw) << 16);
    float r;
    asm("cvt.f32.f16 %0, %1;" : "=f"(r) : "h"(raw));
    return r;
}
// Element `idx` of a gradient block whose elements are fp32 (dtype GAR_F32) or 16 bits wide.
__device__ __forceinline__ float load_elem(const void* g, int64_t idx, int dtype) {
    if (dtype == GAR_F32) return __ldg(static_cast<const float*>(g) + idx);
    return widen16(__ldg(static_cast<const unsigned short*>(g) + idx), dtype);
}

// ---- kernel launchers (one per translation unit) --------------------------
// Pairwise squared distances of n rows over columns [0, d); result in dist[n*n].
// mode: a gar_distance_mode_t.
cudaError_t launch_distances(const float* grads, int n, int64_t d, int64_t ld, double* dist,
                             const Workspace& ws, int sm_count, int mode, cudaStream_t stream);
// The same for 16-bit gradients (dtype GAR_BF16 or GAR_F16; grads points at 2-byte elements).
cudaError_t launch_distances_16(const void* grads, int dtype, int n, int64_t d, int64_t ld, double* dist,
                                const Workspace& ws, int sm_count, cudaStream_t stream);

// Tensor-core variant (tcgen05, accumulators in tensor memory) for 16 < n <= 64 and 16-byte
// aligned rows, used from kMmaMinDim coordinates on.
constexpr int64_t kMmaMinDim = 32768;
cudaError_t launch_distances_umma(const float* grads, int n, int64_t d, int64_t ld, double* dist,
                                  const Workspace& ws, int sm_count, cudaStream_t stream, int dtype = GAR_F32);

// Scoring + iterative selection (and schedule construction) into *sel.
cudaError_t launch_select(int rule, const double* dist, int n, int f, int m, int theta, int beta,
                          int median_of_agr, int even_median, gar_selection_t* sel, cudaStream_t stream, int count = 1);
cudaError_t launch_schedule_only(gar_selection_t* sel, cudaStream_t stream);

// Coordinate phase.
cudaError_t launch_coordinate(const float* grads, int n, int64_t d, int64_t ld,
                              gar_selection_t* sel, int theta, int preagg, const K3Out& out,
                              int sm_count, cudaStream_t stream, int dtype = GAR_F32);

// One warp waits, bounded, on a barrier nobody arrives on; result[0] = status, result[1] = ns.
cudaError_t launch_selftest_wait(unsigned limit, long long* result, cudaStream_t stream);

// Batched launches over device arrays of descriptors: `total_ctas` CTAs, cta_desc[b] = the
// descriptor CTA b works on.  Distances of every tensor into dist + index * n * n (difference
// form: the ring kernel up to 16 rows, the tiled kernel beyond; `vec` = 4, 2, 1: every tensor's
// rows are 16-byte / 8-byte / 4-byte aligned; kMultiStaged: the staged kernel; partial sums at partials + b * kPairSlots, tickets +
// index); coordinate phase of every tensor with the selection
// sel + index * sel_stride (register kernel, `vec` coordinates per thread).
cudaError_t launch_distances_multi(const MultiDesc* desc, const int* cta_desc, int total_ctas, int n, int vec, double* dist,
                                   double* partials, unsigned int* tickets, unsigned int* error_word, int dtype, cudaStream_t stream);
// `vec` of the class of long tensors (n <= 16, 16-byte aligned rows) that go through the staged
// kernel, one CTA per SM; and the length from which a tensor belongs to it
constexpr int kMultiStaged = 8;
constexpr int64_t kMultiStagedMinDim = 32768;
cudaError_t launch_coordinate_multi(const MultiDesc* desc, const int* cta_desc, int total_ctas, int n, int theta, int preagg,
                                    int vec, gar_selection_t* sel, int sel_stride, float lr, float mu, int dtype, cudaStream_t stream);
// Sizes that decide how many CTAs a tensor gets in the batched launches.
int distances_multi_chunk(int n, int vec, int dtype);
int coordinate_multi_threads(int n, int theta, int preagg, int vec);
// The vector width launch_coordinate_multi may be given for a tensor of these addresses and sizes.
int coordinate_multi_vec(const void* grads, const void* out, const void* x, const void* v, int64_t d, int64_t ld, int theta,
                         int preagg, int dtype);

// cudaSuccess -> GAR_OK; anything else is remembered for gar_last_cuda_error and becomes GAR_ERR_CUDA
int cuda_status(cudaError_t err);

}  // namespace gar
