// Pairwise squared l2 distances of n <= 64 gradients of dimension d in ONE
// streaming pass over the n x d block (Algorithm 1, multi-Krum: the distances
// to the k-f-2 closest vectors; the only O(n^2 d) step, computed once).
//
// Layout of the work
//  * Rows are grouped in blocks of 8; a "tile" is a pair of row blocks (I <= J).
//    Off-diagonal tiles hold 64 pairs, diagonal tiles the 28 pairs i < j.
//  * A CTA walks column slabs of TK coordinates (persistent, slab = cta + k*grid).
//    A slab of all rows is staged in shared memory through an NSTAGE-deep ring.
//  * A thread owns one tile and one of 8*G column lanes: it reads 8 + 8 float4
//    from shared memory and updates 64 (or 28) fp32 accumulators in registers,
//    (a-b) then fma -- the difference form, exact to fp32 rounding per term.
//  * fp32 accumulators only ever hold a few dozen terms: every FLUSH slabs they
//    are reduced over the tile's 8 lanes by shuffles and added to fp64 sums in
//    shared memory.  CTA sums go to a global partial array; the last CTA to
//    finish (ticket counter) adds the partials in CTA order in fp64 and writes
//    the symmetric matrix.  No floating-point atomics: results are
//    bit-reproducible and D_ij == D_ji by construction.
#include <cooperative_groups.h>

#include "gar_internal.cuh"

namespace gar {
namespace {

template <int NB> struct K1Shape;
// G = column-lane groups per tile, KQ = float4 passes per slab, FLUSH = slabs per fp64 flush
// NSTAGE = depth of the shared-memory ring
template <> struct K1Shape<1> { static constexpr int G = 32, KQ = 1, FLUSH = 16, NSTAGE = 3; };
template <> struct K1Shape<2> { static constexpr int G = 12, KQ = 1, FLUSH = 16, NSTAGE = 3; };
template <> struct K1Shape<3> { static constexpr int G = 6,  KQ = 1, FLUSH = 16, NSTAGE = 4; };
template <> struct K1Shape<4> { static constexpr int G = 3,  KQ = 2, FLUSH = 8,  NSTAGE = 3; };
template <> struct K1Shape<5> { static constexpr int G = 2,  KQ = 2, FLUSH = 8,  NSTAGE = 4; };
template <> struct K1Shape<6> { static constexpr int G = 2,  KQ = 2, FLUSH = 8,  NSTAGE = 4; };
template <> struct K1Shape<7> { static constexpr int G = 2,  KQ = 2, FLUSH = 8,  NSTAGE = 4; };
template <> struct K1Shape<8> { static constexpr int G = 1,  KQ = 4, FLUSH = 4,  NSTAGE = 4; };

template <int NB> struct K1Dims {
    static constexpr int R      = NB * 8;                    // staged rows (zero padded)
    static constexpr int TILES  = NB * (NB + 1) / 2;
    static constexpr int OFF    = NB * (NB - 1) / 2;         // off-diagonal tiles come first
    static constexpr int G      = K1Shape<NB>::G;
    static constexpr int KQ     = K1Shape<NB>::KQ;
    static constexpr int FLUSH  = K1Shape<NB>::FLUSH;
    static constexpr int NSTAGE = K1Shape<NB>::NSTAGE;
    static constexpr int LANES  = 8 * G;                     // float4 lanes per pass
    static constexpr int TK4    = LANES * KQ;                // float4 per row per slab
    static constexpr int TK     = TK4 * 4;                   // coordinates per slab
    static constexpr int SLOTS  = TILES * G;                 // (tile, group) owners
    static constexpr int ACTIVE = SLOTS * 8;
    static constexpr int THREADS = (ACTIVE + 31) / 32 * 32;
    static constexpr size_t STAGE_BYTES = size_t(R) * TK * 4;
    static constexpr size_t SUM_BYTES   = size_t(SLOTS) * 64 * sizeof(double);
    static constexpr size_t SMEM_BYTES  = NSTAGE * STAGE_BYTES + SUM_BYTES;
};

__device__ __forceinline__ void tile_to_blocks(int p, int nb, int off, int& I, int& J) {
    if (p >= off) { I = J = p - off; return; }
    // off-diagonal tiles enumerated row by row: (0,1),(0,2)..(0,nb-1),(1,2)..
    int i = 0, rem = p;
    while (rem >= nb - 1 - i) { rem -= nb - 1 - i; ++i; }
    I = i; J = i + 1 + rem;
}

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc, int src_bytes) {
    unsigned s = static_cast<unsigned>(__cvta_generic_to_shared(smem_dst));
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(s), "l"(gsrc), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}

// Stage one slab (all R rows, TK columns from t0) into shared memory.
// VEC path: 16-byte cp.async with zero fill past n rows / d columns.
template <int NB, bool VEC>
__device__ __forceinline__ void stage_slab(float* sm, const float* __restrict__ g, int n, int64_t d,
                                           int64_t ld, int64_t t0) {
    using D = K1Dims<NB>;
    if constexpr (VEC) {
        for (int idx = threadIdx.x; idx < D::R * D::TK4; idx += D::THREADS) {
            int row = idx / D::TK4, c4 = idx - row * D::TK4;
            int64_t col = t0 + 4 * int64_t(c4);
            int64_t left = d - col;                       // valid coordinates from col
            int bytes = (row < n && left > 0) ? (left >= 4 ? 16 : int(left) * 4) : 0;
            const float* src = bytes ? g + int64_t(row) * ld + col : g;
            cp_async16(sm + size_t(row) * D::TK + 4 * c4, src, bytes);
        }
    } else {
        for (int idx = threadIdx.x; idx < D::R * D::TK; idx += D::THREADS) {
            int row = idx / D::TK, c = idx - row * D::TK;
            int64_t col = t0 + c;
            float v = (row < n && col < d) ? __ldg(g + int64_t(row) * ld + col) : 0.0f;
            sm[size_t(row) * D::TK + c] = v;
        }
    }
}

template <int NB, bool VEC>
__global__ void __launch_bounds__(K1Dims<NB>::THREADS)
k1_distances(const float* __restrict__ g, int n, int64_t d, int64_t ld, double* __restrict__ dist,
             double* __restrict__ partials, unsigned int* __restrict__ ticket) {
    using D = K1Dims<NB>;
    constexpr int NSTAGE = D::NSTAGE;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float*  stage = reinterpret_cast<float*>(smem_raw);
    double* sums  = reinterpret_cast<double*>(smem_raw + NSTAGE * D::STAGE_BYTES);
    __shared__ int is_last;

    const int tid  = threadIdx.x;
    const int slot = tid >> 3;                 // (group, tile) owner index
    const int c    = tid & 7;                  // lane inside the owner
    const bool active = slot < D::SLOTS;
    const int grp  = active ? slot / D::TILES : 0;
    const int p    = active ? slot - grp * D::TILES : 0;
    int I, J;
    tile_to_blocks(p, NB, D::OFF, I, J);
    const bool diag = (p >= D::OFF);

    for (int i = tid; i < D::SLOTS * 64; i += D::THREADS) sums[i] = 0.0;
    __syncthreads();

    float acc[64];
#pragma unroll
    for (int i = 0; i < 64; ++i) acc[i] = 0.0f;

    const int64_t nslabs = (d + D::TK - 1) / D::TK;
    const int64_t first = blockIdx.x, step = gridDim.x;
    const int64_t mine = first < nslabs ? (nslabs - first + step - 1) / step : 0;

    auto flush = [&]() {
        // reduce each accumulator over the tile's 8 lanes, then lane (pair & 7) adds it in fp64
#pragma unroll
        for (int i = 0; i < 64; ++i) {
            float v = acc[i];
            v += __shfl_xor_sync(0xffffffffu, v, 1);
            v += __shfl_xor_sync(0xffffffffu, v, 2);
            v += __shfl_xor_sync(0xffffffffu, v, 4);
            if (active && (i & 7) == c) sums[slot * 64 + i] += double(v);
            acc[i] = 0.0f;
        }
    };

    if constexpr (VEC) {
        for (int s = 0; s < NSTAGE - 1; ++s) {
            if (s < mine) stage_slab<NB, true>(stage + size_t(s) * D::R * D::TK, g, n, d, ld, (first + s * step) * D::TK);
            cp_async_commit();
        }
    }

    int since_flush = 0;
    for (int64_t it = 0; it < mine; ++it) {
        float* cur;
        if constexpr (VEC) {
            cp_async_wait<NSTAGE - 2>();
            __syncthreads();
            int64_t nxt = it + NSTAGE - 1;
            if (nxt < mine)
                stage_slab<NB, true>(stage + size_t(nxt % NSTAGE) * D::R * D::TK, g, n, d, ld, (first + nxt * step) * D::TK);
            cp_async_commit();
            cur = stage + size_t(it % NSTAGE) * D::R * D::TK;
        } else {
            __syncthreads();
            stage_slab<NB, false>(stage, g, n, d, ld, (first + it * step) * D::TK);
            __syncthreads();
            cur = stage;
        }

        if (active) {
            const float4* s4 = reinterpret_cast<const float4*>(cur);
#pragma unroll
            for (int k = 0; k < D::KQ; ++k) {
                const int q = k * D::LANES + grp * 8 + c;
                float4 a[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) a[i] = s4[(I * 8 + i) * D::TK4 + q];
                if (!diag) {
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const float4 b = s4[(J * 8 + j) * D::TK4 + q];
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            float dx = a[i].x - b.x, dy = a[i].y - b.y, dz = a[i].z - b.z, dw = a[i].w - b.w;
                            float t = acc[i * 8 + j];
                            t = fmaf(dx, dx, t); t = fmaf(dy, dy, t); t = fmaf(dz, dz, t); t = fmaf(dw, dw, t);
                            acc[i * 8 + j] = t;
                        }
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
#pragma unroll
                        for (int j = i + 1; j < 8; ++j) {
                            float dx = a[i].x - a[j].x, dy = a[i].y - a[j].y, dz = a[i].z - a[j].z, dw = a[i].w - a[j].w;
                            float t = acc[i * 8 + j];
                            t = fmaf(dx, dx, t); t = fmaf(dy, dy, t); t = fmaf(dz, dz, t); t = fmaf(dw, dw, t);
                            acc[i * 8 + j] = t;
                        }
                    }
                }
            }
        }
        if (++since_flush == D::FLUSH) { flush(); since_flush = 0; }
    }
    if constexpr (VEC) cp_async_wait<0>();
    flush();
    __syncthreads();

    // CTA partial: sum the groups in order, one fp64 per (tile, pair)
    double* my_partial = partials + size_t(blockIdx.x) * kPairSlots;
    for (int i = tid; i < D::TILES * 64; i += D::THREADS) {
        double s = 0.0;
#pragma unroll 1
        for (int gq = 0; gq < D::G; ++gq) s += sums[(gq * D::TILES + (i >> 6)) * 64 + (i & 63)];
        my_partial[i] = s;
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        unsigned int t = atomicAdd(ticket, 1u);
        is_last = (t == gridDim.x - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();

    // last CTA: add the partials in CTA order and write the symmetric matrix
    for (int i = tid; i < D::TILES * 64; i += D::THREADS) {
        double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
        unsigned b = 0;
        for (; b + 4 <= gridDim.x; b += 4) {
            s0 += __ldcg(partials + size_t(b) * kPairSlots + i);
            s1 += __ldcg(partials + size_t(b + 1) * kPairSlots + i);
            s2 += __ldcg(partials + size_t(b + 2) * kPairSlots + i);
            s3 += __ldcg(partials + size_t(b + 3) * kPairSlots + i);
        }
        for (; b < gridDim.x; ++b) s0 += __ldcg(partials + size_t(b) * kPairSlots + i);
        const double s = (s0 + s1) + (s2 + s3);
        int pi = i >> 6, pr = i & 63, bi, bj;
        tile_to_blocks(pi, NB, D::OFF, bi, bj);
        const int ra = bi * 8 + (pr >> 3), rb = bj * 8 + (pr & 7);
        if (ra < n && rb < n && ra < rb) {
            dist[ra * n + rb] = s;
            dist[rb * n + ra] = s;
        }
    }
    for (int i = tid; i < n; i += D::THREADS) dist[i * n + i] = 0.0;
    if (tid == 0) *ticket = 0u;               // ready for the next call
}

template <int NB, bool VEC>
cudaError_t launch_nb(const float* g, int n, int64_t d, int64_t ld, double* dist, const Workspace& ws,
                      int sm_count, cudaStream_t stream) {
    using D = K1Dims<NB>;
    auto kern = k1_distances<NB, VEC>;
    static int per_sm_cache[64] = {0};        // per device: 0 = not configured yet
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    int per_sm = (dev >= 0 && dev < 64) ? per_sm_cache[dev] : 0;
    if (per_sm == 0) {
        err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(D::SMEM_BYTES));
        if (err != cudaSuccess) return err;
        err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, D::THREADS, D::SMEM_BYTES);
        if (err != cudaSuccess) return err;
        if (per_sm < 1) per_sm = 1;
        if (dev >= 0 && dev < 64) per_sm_cache[dev] = per_sm;
    }
    int64_t nslabs = (d + D::TK - 1) / D::TK;
    int64_t grid = int64_t(sm_count) * per_sm;
    if (grid > kMaxCtasK1) grid = kMaxCtasK1;
    if (grid > nslabs) grid = nslabs;
    kern<<<unsigned(grid), D::THREADS, D::SMEM_BYTES, stream>>>(g, n, d, ld, dist, ws.partials(), ws.ticket());
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_distances(const float* grads, int n, int64_t d, int64_t ld, double* dist,
                             const Workspace& ws, int sm_count, cudaStream_t stream) {
    const bool vec = (reinterpret_cast<uintptr_t>(grads) % 16 == 0) && (ld % 4 == 0);
    const int nb = (n + 7) / 8;
#define GAR_K1_CASE(NBV)                                                                      \
    case NBV:                                                                                 \
        return vec ? launch_nb<NBV, true>(grads, n, d, ld, dist, ws, sm_count, stream)        \
                   : launch_nb<NBV, false>(grads, n, d, ld, dist, ws, sm_count, stream);
    switch (nb) {
        GAR_K1_CASE(1) GAR_K1_CASE(2) GAR_K1_CASE(3) GAR_K1_CASE(4)
        GAR_K1_CASE(5) GAR_K1_CASE(6) GAR_K1_CASE(7) GAR_K1_CASE(8)
    }
#undef GAR_K1_CASE
    return cudaErrorInvalidValue;
}

}  // namespace gar
