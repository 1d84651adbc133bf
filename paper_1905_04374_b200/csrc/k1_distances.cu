// Pairwise squared l2 distances of n <= 64 gradients of dimension d in ONE
// streaming pass over the n x d block (Algorithm 1, multi-Krum: the distances
// to the k-f-2 closest vectors; the only O(n^2 d) step, computed once).
//
// Every pair term is (a-b) then fma in fp32 -- the difference form, exact to
// fp32 rounding per term.  fp32 accumulators only ever hold a few thousand
// terms: they are reduced across lanes by shuffles and added to fp64 sums in
// shared memory.  CTA sums go to a global partial array; the last CTA to finish
// (ticket counter) adds the partials in CTA order in fp64 and writes the
// symmetric matrix.  No floating-point atomics: results are bit-reproducible
// and D_ij == D_ji by construction.
//
// Three kernels:
//  * n <= 16, 16-byte aligned rows, d of at least one tile per SM ("direct, staged"): tiles of
//    1024 coordinates of all n rows arrive in shared memory by one bulk copy per row; a thread
//    reads its four coordinates of every row and updates all n(n-1)/2 accumulators in registers
//    with packed two-lane fp32 instructions.  HBM-bound.
//  * n <= 16 otherwise ("direct"): a thread fetches its V coordinates of all n rows through its
//    own ring of cp.async copies and updates the accumulators with scalar instructions.
//  * n > 16 ("tiled"): rows are grouped in blocks of 8; a column slab of all rows
//    is staged in shared memory through a cp.async ring.  A half-warp owns either
//    one off-diagonal 8x8 tile (64 pairs) or two diagonal tiles (2 x 28 pairs);
//    warps are homogeneous, so every warp runs one code path and all carry about
//    the same work.  Every pair sees the same column-to-lane assignment and the
//    same reduction tree, so identical rows get bit-identical distances.
//    FMA-pipe-bound.
#include <mutex>

#include "gar_internal.cuh"
#include "mbar.cuh"

namespace gar {
namespace {

// ------------------------------------------------------------------ helpers
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc, int src_bytes) {
    unsigned s = static_cast<unsigned>(__cvta_generic_to_shared(smem_dst));
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(s), "l"(gsrc), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}

// Sum of v[i] over the LANES lanes of a lane group (LANES = 8, 16 or 32, groups
// aligned), "reduce-scatter" style: each step exchanges half of the remaining
// values with the partner lane, so the whole reduction costs about COUNT
// shuffles instead of COUNT*log2(LANES).  COUNT must be a multiple of LANES.
// On return v[0 .. COUNT/LANES) of lane l holds the totals of the indices
// scatter_base<COUNT, LANES>(l) + (0 .. COUNT/LANES).
template <int COUNT, int LANES>
__device__ __forceinline__ void reduce_scatter(float (&v)[COUNT], int lane) {
    int len = COUNT;
#pragma unroll
    for (int m = LANES / 2; m >= 1; m >>= 1) {
        const int half = len / 2;
        const bool upper = (lane & m) != 0;
#pragma unroll
        for (int i = 0; i < COUNT / 2; ++i) {
            if (i < half) {
                const float lo = v[i], hi = v[i + half];
                const float send = upper ? lo : hi, keep = upper ? hi : lo;
                v[i] = keep + __shfl_xor_sync(0xffffffffu, send, m);
            }
        }
        len = half;
    }
}
template <int COUNT, int LANES> __device__ __forceinline__ int scatter_base(int lane) {
    int base = 0, len = COUNT;
#pragma unroll
    for (int m = LANES / 2; m >= 1; m >>= 1) {
        len /= 2;
        if (lane & m) base += len;
    }
    return base;
}

// Last-CTA reduction of the per-CTA partial sums (fixed order) -> `combine(slot, sum)`.
template <typename F>
__device__ __forceinline__ void reduce_partials(const double* partials, int nslots, int nthreads, unsigned nctas, F combine) {
    for (int i = threadIdx.x; i < nslots; i += nthreads) {
        double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
        unsigned b = 0;
        for (; b + 4 <= nctas; b += 4) {
            s0 += __ldcg(partials + size_t(b) * kPairSlots + i);
            s1 += __ldcg(partials + size_t(b + 1) * kPairSlots + i);
            s2 += __ldcg(partials + size_t(b + 2) * kPairSlots + i);
            s3 += __ldcg(partials + size_t(b + 3) * kPairSlots + i);
        }
        for (; b < nctas; ++b) s0 += __ldcg(partials + size_t(b) * kPairSlots + i);
        combine(i, (s0 + s1) + (s2 + s3));
    }
}

// Returns true in exactly one of the `nctas` CTAs that share the ticket: the last one to arrive.
// All of this CTA's partial sums must have been written before the call.
__device__ __forceinline__ bool last_cta_ticket(unsigned int* ticket, unsigned nctas) {
    __shared__ int is_last;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) is_last = (atomicAdd(ticket, 1u) == nctas - 1);
    __syncthreads();
    if (is_last) __threadfence();
    return is_last != 0;
}

// ---- pieces the two direct kernels (n <= 16) share
// The arithmetic.  Rows are taken two at a time: R_a = (x_2a, x_2a+1) sits in one 64-bit register
// pair, and one packed subtract plus one packed multiply-add (sub.f32x2, fma.rn.f32x2: two IEEE
// fp32 operations each, one issue slot) serve two pairs at once --
//     R_a - R_b          -> pairs (2a, 2b), (2a+1, 2b+1)
//     R_a - swap(R_b)    -> pairs (2a, 2b+1), (2a+1, 2b)
//     R_a - (x_N-1, x_N-1) for the unpaired last row of an odd N
// and the pair (2a, 2a+1) inside a row pair takes scalar instructions: 112 issue slots per
// coordinate for 15 rows instead of 210.
template <int N> struct K1Pairs {
    static constexpr int NP = N * (N - 1) / 2;
    static constexpr int NPAD = (NP + 31) / 32 * 32;
    static constexpr int NF = N / 2;                               // whole row pairs
    static constexpr int NBLK = NF * (NF - 1) / 2;                 // blocks of two row pairs
    static constexpr int NPK = 2 * NBLK + (N % 2 ? NF : 0);        // packed accumulators
    static_assert(2 * NPK + NF == NP, "accumulator slots");
};

__device__ __forceinline__ unsigned long long pack2(float lo, float hi) {
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(unsigned long long p, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(p));
}
// acc += (a - b)^2 in both lanes
__device__ __forceinline__ void sqdiff2(unsigned long long& acc, unsigned long long a, unsigned long long b) {
    unsigned long long df;
    asm("sub.f32x2 %0, %1, %2;" : "=l"(df) : "l"(a), "l"(b));
    asm("fma.rn.f32x2 %0, %1, %1, %0;" : "+l"(acc) : "l"(df));
}

// The accumulators of one thread.  Slot order (the order of the CTA's partial sums):
//   for a < b < NF:   4 * blk(a, b) + {0: (2a, 2b), 1: (2a+1, 2b+1), 2: (2a, 2b+1), 3: (2a+1, 2b)}
//   odd N, a < NF:    4 * NBLK + 2a + {0: (2a, N-1), 1: (2a+1, N-1)}
//   a < NF:           2 * NPK + a: (2a, 2a+1)
template <int N> struct K1BAcc {
    using S = K1Pairs<N>;
    unsigned long long pk[S::NPK > 0 ? S::NPK : 1];
    float dg[S::NF > 0 ? S::NF : 1];

    __device__ __forceinline__ void zero() {
#pragma unroll
        for (int i = 0; i < S::NPK; ++i) pk[i] = 0ull;
#pragma unroll
        for (int i = 0; i < S::NF; ++i) dg[i] = 0.0f;
    }
    // one coordinate of all rows
    __device__ __forceinline__ void add(const float (&x)[N]) {
        unsigned long long R[S::NF > 0 ? S::NF : 1];
#pragma unroll
        for (int a = 0; a < S::NF; ++a) R[a] = pack2(x[2 * a], x[2 * a + 1]);
        int k = 0;
#pragma unroll
        for (int a = 0; a < S::NF; ++a) {
#pragma unroll
            for (int b = a + 1; b < S::NF; ++b) {
                sqdiff2(pk[k], R[a], R[b]);
                sqdiff2(pk[k + 1], R[a], pack2(x[2 * b + 1], x[2 * b]));
                k += 2;
            }
        }
        if constexpr (N % 2 == 1) {
            const unsigned long long last = pack2(x[N - 1], x[N - 1]);
#pragma unroll
            for (int a = 0; a < S::NF; ++a) sqdiff2(pk[2 * S::NBLK + a], R[a], last);
        }
#pragma unroll
        for (int a = 0; a < S::NF; ++a) { const float df = x[2 * a] - x[2 * a + 1]; dg[a] = fmaf(df, df, dg[a]); }
    }
    // the warp's fp32 accumulators -> its fp64 sums in shared memory (fixed shuffle tree), then zero
    __device__ __forceinline__ void flush(double* warp_sums, int lane, int sbase) {
        float flat[S::NPAD];
#pragma unroll
        for (int i = 0; i < S::NPK; ++i) unpack2(pk[i], flat[2 * i], flat[2 * i + 1]);
#pragma unroll
        for (int i = 0; i < S::NF; ++i) flat[2 * S::NPK + i] = dg[i];
#pragma unroll
        for (int i = S::NP; i < S::NPAD; ++i) flat[i] = 0.0f;
        reduce_scatter<S::NPAD, 32>(flat, lane);
#pragma unroll
        for (int i = 0; i < S::NPAD / 32; ++i) warp_sums[sbase + i] += double(flat[i]);
        zero();
    }
};
// slot of K1BAcc -> the pair of rows (i < j)
template <int N> __device__ __forceinline__ void k1b_slot_rows(int slot, int& i, int& j) {
    using S = K1Pairs<N>;
    if (slot >= 2 * S::NPK) { i = 2 * (slot - 2 * S::NPK); j = i + 1; return; }
    if (slot >= 4 * S::NBLK) { i = slot - 4 * S::NBLK; j = N - 1; return; }
    int blk = slot >> 2, a = 0;
    while (blk >= S::NF - 1 - a) { blk -= S::NF - 1 - a; ++a; }
    const int b = a + 1 + blk, which = slot & 3;
    i = 2 * a + (which & 1);
    j = 2 * b + ((which == 1 || which == 2) ? 1 : 0);
}

// ---- the ring kernel's scalar form of the same sums (it is bound by the latency of its copies, and
// the packed form costs it registers it needs for three CTAs per SM: measured 2.5 times slower there)
// acc[p] += sum_v (x[i][v] - x[j][v])^2 over the pairs p = (0,1), (0,2), .., (0,N-1), (1,2), ..
template <int N, int V, int NPAD>
__device__ __forceinline__ void direct_pairs(const float (&x)[N][V], float (&acc)[NPAD]) {
    int p = 0;
#pragma unroll
    for (int i = 0; i < N; ++i) {
#pragma unroll
        for (int j = i + 1; j < N; ++j) {
            float t = acc[p];
#pragma unroll
            for (int v = 0; v < V; ++v) { const float df = x[i][v] - x[j][v]; t = fmaf(df, df, t); }
            acc[p] = t;
            ++p;
        }
    }
}
// One coordinate t of all rows straight from global memory (ragged ends).
template <int N, int NPAD>
__device__ __forceinline__ void direct_tail_coordinate(const void* __restrict__ g, int64_t ld, int64_t t, float (&acc)[NPAD],
                                                       int dtype = GAR_F32) {
    float x[N][1];
#pragma unroll
    for (int r = 0; r < N; ++r) x[r][0] = load_elem(g, int64_t(r) * ld + t, dtype);
    direct_pairs<N, 1, NPAD>(x, acc);
}
// The warp's fp32 accumulators -> its fp64 sums in shared memory (fixed shuffle tree), then zero.
template <int NPAD>
__device__ __forceinline__ void direct_flush(float (&acc)[NPAD], double* warp_sums, int lane, int sbase) {
    reduce_scatter<NPAD, 32>(acc, lane);
#pragma unroll
    for (int i = 0; i < NPAD / 32; ++i) warp_sums[sbase + i] += double(acc[i]);
#pragma unroll
    for (int i = 0; i < NPAD; ++i) acc[i] = 0.0f;
}
// Pair index p of direct_pairs -> (i, j).
template <int N> __device__ __forceinline__ void direct_pair_rows(int p, int& i, int& j) {
    i = 0;
    int rem = p;
    while (rem >= N - 1 - i) { rem -= N - 1 - i; ++i; }
    j = i + 1 + rem;
}

// ======================================================== direct kernel, n <= 16
constexpr int K1R_THREADS = 128;
constexpr int K1R_FLUSH = 64;       // iterations between fp64 flushes
constexpr int K1R_STAGES = 4;       // depth of the per-thread cp.async ring
constexpr int K1B_V = 4;            // staged kernel: coordinates per thread and tile (two: 35 % slower, the per-tile barrier shows) // staged kernel: rows from which a thread owns two coordinates instead of four

template <int BYTES>
__device__ __forceinline__ void cp_async_small(void* smem_dst, const void* gsrc) {
    unsigned s = static_cast<unsigned>(__cvta_generic_to_shared(smem_dst));
    if constexpr (BYTES == 16) asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gsrc) : "memory");
    else asm volatile("cp.async.ca.shared.global [%0], [%1], %2;\n" ::"r"(s), "l"(gsrc), "n"(BYTES) : "memory");
}

template <int N, int V> struct K1RDims {
    static constexpr size_t RING_BYTES = size_t(K1R_STAGES) * N * K1R_THREADS * V * sizeof(float);
};

// Each thread owns V coordinates of all N rows per iteration.  The rows travel
// through a ring of cp.async copies into shared-memory slots private to the
// thread (K1R_STAGES - 1 iterations in flight, no barrier, no register staging),
// so many bytes are in flight per SM while the registers hold the accumulators.
// bx, gx: this CTA's place among the CTAs that share the problem (the ticket, the partial sums);
// path_word may be null.
template <int N, int V>
__device__ __forceinline__ void k1_direct_body(const float* __restrict__ g, const int64_t d, const int64_t ld, double* __restrict__ dist,
                                               double* __restrict__ partials, unsigned int* __restrict__ ticket,
                                               unsigned int* __restrict__ path_word, const unsigned bx, const unsigned gx) {
    constexpr int NP = K1Pairs<N>::NP, NPAD = K1Pairs<N>::NPAD;
    constexpr int WARPS = K1R_THREADS / 32;
    extern __shared__ __align__(16) float ring[];            // [stage][row][thread][V]
    __shared__ double sums[WARPS][NPAD];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int i = tid; i < WARPS * NPAD; i += K1R_THREADS) (&sums[0][0])[i] = 0.0;
    __syncthreads();

    float acc[NPAD];
#pragma unroll
    for (int i = 0; i < NPAD; ++i) acc[i] = 0.0f;
    const int sbase = scatter_base<NPAD, 32>(lane);

    auto flush = [&]() { direct_flush<NPAD>(acc, sums[warp], lane, sbase); };
    // request the rows of vector index vi into ring stage st (zeros past the end)
    auto request = [&](int st, int64_t vi, bool valid) {
        float* slot = ring + (size_t(st) * N * K1R_THREADS + tid) * V;
#pragma unroll
        for (int r = 0; r < N; ++r) {
            float* dst = slot + size_t(r) * K1R_THREADS * V;
            if (valid) {
                cp_async_small<4 * V>(dst, g + int64_t(r) * ld + vi * V);
            } else {
#pragma unroll
                for (int v = 0; v < V; ++v) dst[v] = 0.0f;
            }
        }
    };
    auto consume = [&](int st) {
        const float* slot = ring + (size_t(st) * N * K1R_THREADS + tid) * V;
        float x[N][V];
#pragma unroll
        for (int r = 0; r < N; ++r) {
            const float* src = slot + size_t(r) * K1R_THREADS * V;
            if constexpr (V == 4) { float4 q = *reinterpret_cast<const float4*>(src); x[r][0] = q.x; x[r][1] = q.y; x[r][2] = q.z; x[r][3] = q.w; }
            else if constexpr (V == 2) { float2 q = *reinterpret_cast<const float2*>(src); x[r][0] = q.x; x[r][1] = q.y; }
            else { x[r][0] = *src; }
        }
        direct_pairs<N, V, NPAD>(x, acc);
    };

    // the loop bound is per warp, so that the flush (warp-collective) is uniform
    const int64_t nvec = d / V;
    const int64_t stride = int64_t(gx) * K1R_THREADS;
    const int64_t wfirst = int64_t(bx) * K1R_THREADS + warp * 32;
    const int64_t iters = wfirst < nvec ? (nvec - wfirst + stride - 1) / stride : 0;
#pragma unroll
    for (int s = 0; s < K1R_STAGES - 1; ++s) {
        if (s < iters) { const int64_t vi = wfirst + s * stride + lane; request(s, vi, vi < nvec); }
        cp_async_commit();
    }
    int since = 0;
    for (int64_t it = 0; it < iters; ++it) {
        cp_async_wait<K1R_STAGES - 2>();
        const int64_t nx = it + K1R_STAGES - 1;
        if (nx < iters) { const int64_t vi = wfirst + nx * stride + lane; request(int(nx % K1R_STAGES), vi, vi < nvec); }
        cp_async_commit();
        consume(int(it % K1R_STAGES));
        if (++since == K1R_FLUSH) { flush(); since = 0; }
    }
    cp_async_wait<0>();
    // ragged tail: the last d % V coordinates, one thread
    if (V > 1 && bx == 0 && tid == 0) {
        for (int64_t t = nvec * V; t < d; ++t) direct_tail_coordinate<N, NPAD>(g, ld, t, acc);
    }
    __syncwarp();
    flush();
    __syncthreads();

    double* my_partial = partials + size_t(bx) * kPairSlots;
    for (int i = tid; i < NP; i += K1R_THREADS) {
        double s = 0.0;
#pragma unroll
        for (int w = 0; w < WARPS; ++w) s += sums[w][i];
        my_partial[i] = s;
    }
    if (!last_cta_ticket(ticket, gx)) return;
    reduce_partials(partials, NP, K1R_THREADS, gx, [&](int p, double s) {
        int i, j;
        direct_pair_rows<N>(p, i, j);
        dist[i * N + j] = s;
        dist[j * N + i] = s;
    });
    for (int i = tid; i < N; i += K1R_THREADS) dist[i * N + i] = 0.0;
    if (tid == 0) {
        *ticket = 0u;                             // ready for the next call
        if (path_word != nullptr) *path_word = kPathDifference;
    }
}

template <int N, int V>
__global__ void __launch_bounds__(K1R_THREADS)
k1_direct(const float* __restrict__ g, int64_t d, int64_t ld, double* __restrict__ dist,
          double* __restrict__ partials, unsigned int* __restrict__ ticket, unsigned int* __restrict__ path_word) {
    k1_direct_body<N, V>(g, d, ld, dist, partials, ticket, path_word, blockIdx.x, gridDim.x);
}
// Batch mode: CTA b works on the tensor of descriptor multi[cta_desc[b]].
template <int N, int V>
__global__ void __launch_bounds__(K1R_THREADS)
k1_direct_multi(const MultiDesc* __restrict__ multi, const int* __restrict__ cta_desc, double* __restrict__ dist,
                double* __restrict__ partials, unsigned int* __restrict__ tickets) {
    const MultiDesc t = multi[cta_desc[blockIdx.x]];
    k1_direct_body<N, V>(static_cast<const float*>(t.grads), t.d, t.ld, dist + size_t(t.index) * N * N,
                         partials + size_t(t.cta_first) * kPairSlots, tickets + t.index, nullptr,
                         blockIdx.x - unsigned(t.cta_first), unsigned(t.ctas));
}

// ================================================ direct kernel, n <= 16, rows staged by bulk copies
// Same differences and sums as k1_direct; the rows travel and the arithmetic issues differently.
//
// Staging.  A tile is TC consecutive coordinates of all N rows; warp 0 fetches it with one bulk
// copy per row (contiguous, 2 or 4 KB of fp32) into a ring of shared-memory stages whose mbarriers
// count the bytes in.  Copies of that size keep HBM busier than 16-byte requests per thread do.
// All eight warps compute, so that every thread may hold up to 255 registers (a ninth warp would
// put three warps on one scheduler, whose 16 K registers then allow 168 per thread: too few for the
// 105 to 120 accumulators of 15 or 16 rows next to the rows themselves).  The warps meet in a named
// barrier once per tile; a warp that has passed it has finished the previous tile, so warp 0 refills
// that tile's stage right behind the barrier and no second set of mbarriers is needed.  (Letting
// every warp wait on the tiles' mbarriers by itself, with a second set to hand stages back, so that
// the warps may drift apart, measured 8 % slower.)
//
// Arithmetic.  Rows are taken two at a time: R_a = (x_2a, x_2a+1) sits in one 64-bit register pair,
// and one packed subtract plus one packed multiply-add (sub.f32x2, fma.rn.f32x2: two IEEE fp32
// operations each, one issue slot) serve two pairs at once --
//     R_a - R_b          -> pairs (2a, 2b), (2a+1, 2b+1)
//     R_a - swap(R_b)    -> pairs (2a, 2b+1), (2a+1, 2b)
//     R_a - (x_N-1, x_N-1) for the unpaired last row of an odd N
// and the pair (2a, 2a+1) inside a row pair takes scalar instructions.  That is 112 issue slots per
// coordinate for 15 rows instead of 210, which is what lets eight warps keep up with HBM.
//
// Needs 16-byte aligned rows (base address and row stride); coordinates after the last whole tile
// are added by CTA 0 with plain loads.  A wait that gives up (bounded) raises the CTA's error slot:
// the last CTA then fills the matrix, diagonal included, with NaN and sets the workspace's error word.
template <int N> struct K1BShape {
    static constexpr int V = K1B_V;                                // coordinates per thread and tile
    static constexpr int THREADS = 256;
    static constexpr int WARPS = THREADS / 32;
    static constexpr int TC = THREADS * V;                         // coordinates per tile
    static constexpr int ROW_BYTES = TC * 4;                       // one fp32 row of a tile
    static constexpr int STAGE_BYTES = N * ROW_BYTES;
    static constexpr int NP = K1Pairs<N>::NP, NPAD = K1Pairs<N>::NPAD;
    static constexpr int SUM_BYTES = WARPS * NPAD * 8;
    static constexpr int STAGES_FIT = (200 * 1024 - SUM_BYTES) / STAGE_BYTES;
    static constexpr int STAGES = STAGES_FIT > 8 ? 8 : STAGES_FIT; // depth of the ring
    static_assert(STAGES >= 3, "ring depth");
};
constexpr int K1B_MIN_TC = 256 * K1B_V;        // coordinates per tile (dispatch threshold)
constexpr int K1B_BAR_COMPUTE = 1;

// dtype: the gradients' element type (gar_dtype_t).  16-bit elements are staged as they are (a row of
// a tile is then half as long) and widened to fp32 when the compute threads read them.
// bx, gx: this CTA's place among the CTAs that share the problem; path_word may be null.
template <int N>
__device__ __forceinline__ void k1_direct_bulk_body(const void* __restrict__ g, const int dtype, const int64_t d, const int64_t ld,
                                                    double* __restrict__ dist, double* __restrict__ partials,
                                                    unsigned int* __restrict__ ticket, unsigned int* __restrict__ error_word,
                                                    unsigned int* __restrict__ path_word, const unsigned bx, const unsigned gx) {
    using S = K1BShape<N>;
    constexpr int NP = S::NP, NPAD = S::NPAD, V = S::V, THREADS = S::THREADS, WARPS = S::WARPS, TC = S::TC, STAGES = S::STAGES;
    const int esize = dtype == GAR_F32 ? 4 : 2;
    const unsigned row_bytes = unsigned(TC) * unsigned(esize);
    const unsigned stage_bytes = unsigned(N) * row_bytes;
    extern __shared__ __align__(128) unsigned char stages[];          // [stage][row][TC elements]
    __shared__ double sums[WARPS][NPAD];
    __shared__ unsigned long long full[STAGES];
    __shared__ int error_flag;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int i = tid; i < WARPS * NPAD; i += THREADS) (&sums[0][0])[i] = 0.0;
    if (tid == 0) {
        for (int st = 0; st < STAGES; ++st) kb_init(&full[st], 1u);
        error_flag = 0;
        kb_fence_init();
    }
    __syncthreads();
    volatile int* error = &error_flag;

    const int64_t ntiles = d / TC;
    const int64_t first = bx, step = gx;
    const int64_t mine = first < ntiles ? (ntiles - first + step - 1) / step : 0;

    // warp 0, lane r fetches row r of this CTA's tile number i into stage i % STAGES
    auto fetch = [&](int64_t i) {
        const int st = int(i % STAGES);
        const unsigned bar = kb_smem_u32(&full[st]);
        if (lane == 0) kb_expect_tx(bar, stage_bytes);
        __syncwarp();
        if (lane < N)
            kb_bulk_load(kb_smem_u32(stages) + unsigned(st) * stage_bytes + unsigned(lane) * row_bytes,
                         static_cast<const char*>(g) + (int64_t(lane) * ld + (first + i * step) * TC) * esize, row_bytes, bar);
    };
    int64_t issued = 0;                              // warp 0: tiles requested so far
    if (warp == 0) {
        for (; issued < STAGES - 1 && issued < mine; ++issued) fetch(issued);
    }

    K1BAcc<N> acc;
    acc.zero();
    const int sbase = scatter_base<NPAD, 32>(lane);
    int st = 0, since = 0;
    unsigned parity = 0;
    int64_t it = 0;
    for (; it < mine; ++it) {
        // one warp waits on the stage's barrier, the others sleep in a hardware barrier meanwhile
        if (warp == 0) kb_wait(kb_smem_u32(&full[st]), parity, error);
        unsigned failed;                          // the same answer in every thread
        asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.b32 q, %1, 0;\n\tbar.red.or.pred p, %2, %3, q;\n\tselp.b32 %0, 1, 0, p;\n\t}"
                     : "=r"(failed) : "r"(*error), "r"(K1B_BAR_COMPUTE), "r"(THREADS) : "memory");
        if (failed) break;
        // every warp is past tile it - 1: its stage takes tile it + STAGES - 1
        if (warp == 0 && issued < mine) { fetch(issued); ++issued; }
        const unsigned char* tile = stages + size_t(st) * stage_bytes;
        if (dtype == GAR_F32) {
#pragma unroll
            for (int v = 0; v < V; ++v) {
                float x[N];
#pragma unroll
                for (int r = 0; r < N; ++r) x[r] = reinterpret_cast<const float*>(tile + size_t(r) * row_bytes)[v * THREADS + tid];
                acc.add(x);
            }
        } else {
#pragma unroll
            for (int v = 0; v < V; v += 2) {
                float x0[N], x1[N];
#pragma unroll
                for (int r = 0; r < N; ++r) {
                    const unsigned q = reinterpret_cast<const unsigned*>(tile + size_t(r) * row_bytes)[(v / 2) * THREADS + tid];
                    x0[r] = widen16(static_cast<unsigned short>(q & 0xffffu), dtype);
                    x1[r] = widen16(static_cast<unsigned short>(q >> 16), dtype);
                }
                acc.add(x0);
                acc.add(x1);
            }
        }
        if (++since == K1R_FLUSH) { acc.flush(sums[warp], lane, sbase); since = 0; }
        if (++st == STAGES) { st = 0; parity ^= 1u; }
    }
    // no copy may be in flight when the CTA leaves: after a failure, wait (bounded) for the tiles
    // that were requested and not consumed
    if (warp == 0) {
        for (int64_t j = it; j < issued; ++j)
            kb_wait(kb_smem_u32(&full[j % STAGES]), unsigned(j / STAGES) & 1u, error, true);
    }
    // coordinates after the last whole tile: CTA 0, plain loads
    if (bx == 0) {
        for (int64_t t = ntiles * TC + tid; t < d; t += THREADS) {
            float x[N];
#pragma unroll
            for (int r = 0; r < N; ++r) x[r] = load_elem(g, int64_t(r) * ld + t, dtype);
            acc.add(x);
        }
    }
    __syncwarp();
    acc.flush(sums[warp], lane, sbase);
    __syncthreads();

    double* my_partial = partials + size_t(bx) * kPairSlots;
    for (int i = tid; i < NP; i += THREADS) {
        double s = 0.0;
#pragma unroll
        for (int w = 0; w < WARPS; ++w) s += sums[w][i];
        my_partial[i] = s;
    }
    if (tid == 0) my_partial[kSlotError] = double(error_flag);
    if (!last_cta_ticket(ticket, gx)) return;
    __shared__ int any_error;
    if (tid == 0) {
        unsigned err = 0u;
        for (unsigned b = 0; b < gx; ++b) err |= unsigned(__ldcg(partials + size_t(b) * kPairSlots + kSlotError));
        any_error = int(err);
        if (err) *error_word = 1u;
    }
    __syncthreads();
    const bool failed = any_error != 0;
    const double nan = __longlong_as_double(0x7ff8000000000000ll);
    reduce_partials(partials, NP, THREADS, gx, [&](int p, double s) {
        int i, j;
        k1b_slot_rows<N>(p, i, j);
        if (failed) s = nan;
        dist[i * N + j] = s;
        dist[j * N + i] = s;
    });
    // a NaN diagonal tells the selection kernel that the matrix is not to be used
    for (int i = tid; i < N; i += THREADS) dist[i * N + i] = failed ? nan : 0.0;
    if (tid == 0) {
        *ticket = 0u;                             // ready for the next call
        if (path_word != nullptr) *path_word = kPathDifference;
    }
}

template <int N>
__global__ void __launch_bounds__(K1BShape<N>::THREADS, 1)
k1_direct_bulk(const void* __restrict__ g, int dtype, int64_t d, int64_t ld, double* __restrict__ dist,
               double* __restrict__ partials, unsigned int* __restrict__ ticket, unsigned int* __restrict__ error_word,
               unsigned int* __restrict__ path_word) {
    k1_direct_bulk_body<N>(g, dtype, d, ld, dist, partials, ticket, error_word, path_word, blockIdx.x, gridDim.x);
}
// Batch mode: CTA b works on the tensor of descriptor multi[cta_desc[b]].
template <int N>
__global__ void __launch_bounds__(K1BShape<N>::THREADS, 1)
k1_direct_bulk_multi(const MultiDesc* __restrict__ multi, const int* __restrict__ cta_desc, double* __restrict__ dist,
                     double* __restrict__ partials, unsigned int* __restrict__ tickets, unsigned int* __restrict__ error_word,
                     int dtype) {
    const MultiDesc t = multi[cta_desc[blockIdx.x]];
    k1_direct_bulk_body<N>(t.grads, dtype, t.d, t.ld, dist + size_t(t.index) * N * N, partials + size_t(t.cta_first) * kPairSlots,
                           tickets + t.index, error_word, nullptr, blockIdx.x - unsigned(t.cta_first), unsigned(t.ctas));
}

// ========================================================= tiled kernel, n > 16
template <int NB> struct K1Shape;
// G = column groups per CTA, KQ = float4 passes of an off-diagonal lane per slab,
// FLUSH = slabs between fp64 flushes, NSTAGE = depth of the shared-memory ring
template <> struct K1Shape<1> { static constexpr int G = 4, KQ = 2, FLUSH = 8, NSTAGE = 3; };   // n <= 16: 16-bit gradients only
template <> struct K1Shape<2> { static constexpr int G = 4, KQ = 2, FLUSH = 8, NSTAGE = 3; };
template <> struct K1Shape<3> { static constexpr int G = 2, KQ = 2, FLUSH = 8, NSTAGE = 3; };
template <> struct K1Shape<4> { static constexpr int G = 2, KQ = 2, FLUSH = 8, NSTAGE = 3; };
template <> struct K1Shape<5> { static constexpr int G = 1, KQ = 2, FLUSH = 8, NSTAGE = 4; };
template <> struct K1Shape<6> { static constexpr int G = 1, KQ = 4, FLUSH = 4, NSTAGE = 3; };
template <> struct K1Shape<7> { static constexpr int G = 1, KQ = 4, FLUSH = 4, NSTAGE = 3; };
template <> struct K1Shape<8> { static constexpr int G = 1, KQ = 2, FLUSH = 8, NSTAGE = 4; };

template <int NB> struct K1Dims {
    static constexpr int R       = NB * 8;                   // staged rows (zero padded)
    static constexpr int OFFJ    = NB * (NB - 1) / 2;        // off-diagonal tiles, half-warp each
    static constexpr int DIAGJ   = (NB + 1) / 2;             // pairs of diagonal tiles, half-warp each
    static constexpr int OFFW    = (OFFJ + 1) / 2;           // warps of off-diagonal tiles per group
    static constexpr int DIAGW   = (DIAGJ + 1) / 2;          // warps of diagonal-tile pairs per group
    static constexpr int GW      = OFFW + DIAGW;             // warps per group
    static constexpr int G       = K1Shape<NB>::G;
    static constexpr int KQ      = K1Shape<NB>::KQ;
    static constexpr int FLUSH   = K1Shape<NB>::FLUSH;
    static constexpr int NSTAGE  = K1Shape<NB>::NSTAGE;
    static constexpr int GQ      = 16 * KQ;                  // float4 columns per group per slab
    static constexpr int TK4     = G * GQ;                   // float4 per row per slab
    static constexpr int TK      = TK4 * 4;                  // coordinates per slab
    static constexpr int THREADS = G * GW * 32;
    static constexpr int TILES   = OFFJ + DIAGJ;             // tile t < OFFJ: off-diagonal
    static constexpr size_t STAGE_BYTES = size_t(R) * TK * 4;
    static constexpr size_t SUM_BYTES   = size_t(G) * TILES * 64 * sizeof(double);
    static constexpr size_t SMEM_BYTES  = NSTAGE * STAGE_BYTES + SUM_BYTES;
    // two CTAs per SM where registers (<= 128 per thread) and shared memory allow it
    static constexpr int MIN_CTAS = (THREADS <= 256 && SMEM_BYTES <= 110 * 1024) ? 2 : 1;
};

__device__ __forceinline__ void off_tile_blocks(int p, int nb, int& I, int& J) {
    // off-diagonal tiles enumerated row by row: (0,1),(0,2)..(0,nb-1),(1,2)..
    int i = 0, rem = p;
    while (rem >= nb - 1 - i) { rem -= nb - 1 - i; ++i; }
    I = i; J = i + 1 + rem;
}

// Stage one slab (all R rows, TK columns from t0) into shared memory.
// VEC path: 16-byte cp.async with zero fill past n rows / d columns.
// ES: bytes per staged element.  4: fp32 (VEC or scalar path; the scalar path widens 16-bit
// elements as it stages them).  2 (VEC only): 16-bit elements staged as they are, 8 per 16-byte copy,
// and widened when the compute loop reads them.
template <int NB, bool VEC, int ES = 4>
__device__ __forceinline__ void stage_slab(float* sm, const float* __restrict__ g, int n, int64_t d,
                                           int64_t ld, int64_t t0, int dtype = GAR_F32) {
    using D = K1Dims<NB>;
    if constexpr (VEC) {
        constexpr int EPC = 16 / ES;                      // elements per 16-byte copy
        constexpr int CPR = D::TK / EPC;                  // copies per row
        for (int idx = threadIdx.x; idx < D::R * CPR; idx += D::THREADS) {
            const int row = idx / CPR, cc = idx - row * CPR;
            const int64_t col = t0 + EPC * int64_t(cc);
            const int64_t left = d - col;                 // valid coordinates from col
            const int bytes = (row < n && left > 0) ? (left >= EPC ? 16 : int(left) * ES) : 0;
            const char* src = bytes ? reinterpret_cast<const char*>(g) + (int64_t(row) * ld + col) * ES : reinterpret_cast<const char*>(g);
            cp_async16(reinterpret_cast<char*>(sm) + (size_t(row) * D::TK + EPC * cc) * ES, src, bytes);
        }
    } else {
        for (int idx = threadIdx.x; idx < D::R * D::TK; idx += D::THREADS) {
            const int row = idx / D::TK, c = idx - row * D::TK;
            const int64_t col = t0 + c;
            sm[size_t(row) * D::TK + c] = (row < n && col < d) ? load_elem(g, int64_t(row) * ld + col, dtype) : 0.0f;   // widened here
        }
    }
}

// Four staged columns (index in units of four columns) as fp32.
template <int ES> __device__ __forceinline__ float4 tile_ld4(const float* tile, int idx4, int dtype) {
    if constexpr (ES == 4) {
        return reinterpret_cast<const float4*>(tile)[idx4];
    } else {
        const uint2 u = reinterpret_cast<const uint2*>(tile)[idx4];
        return make_float4(widen16(static_cast<unsigned short>(u.x & 0xffffu), dtype), widen16(static_cast<unsigned short>(u.x >> 16), dtype),
                           widen16(static_cast<unsigned short>(u.y & 0xffffu), dtype), widen16(static_cast<unsigned short>(u.y >> 16), dtype));
    }
}

// bx, gx: this CTA's place among the CTAs that share the problem; path_word may be null.
template <int NB, bool VEC, int ES>
__device__ __forceinline__ void k1_tiled_body(const float* __restrict__ g, const int n, const int64_t d, const int64_t ld,
                                              double* __restrict__ dist, double* __restrict__ partials,
                                              unsigned int* __restrict__ ticket, unsigned int* __restrict__ path_word,
                                              const int dtype, const unsigned bx, const unsigned gx) {
    using D = K1Dims<NB>;
    constexpr int NSTAGE = D::NSTAGE;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float*  stage = reinterpret_cast<float*>(smem_raw);
    double* sums  = reinterpret_cast<double*>(smem_raw + NSTAGE * D::STAGE_BYTES);   // [G][TILES][64]

    const int tid = threadIdx.x, lane = tid & 31;
    const int warp = tid >> 5;
    const int grp = warp / D::GW, gw = warp - grp * D::GW;
    const bool off_warp = gw < D::OFFW;
    // a half-warp per job: an off-diagonal tile (I, J), or the diagonal tiles I and J = I + 1
    int tile, I = 0, J = 0;
    bool active;
    const int c = lane & 15;
    if (off_warp) {
        const int job = gw * 2 + (lane >> 4);
        active = job < D::OFFJ;
        tile = active ? job : 0;
        off_tile_blocks(tile, NB, I, J);
    } else {
        const int job = (gw - D::OFFW) * 2 + (lane >> 4);
        active = job < D::DIAGJ;
        I = active ? 2 * job : 0;
        J = (I + 1 < NB) ? I + 1 : I;          // odd block count: the last job repeats its tile (ignored later)
        tile = D::OFFJ + (active ? job : 0);
    }
    double* my_sums = sums + (size_t(grp) * D::TILES + tile) * 64;

    for (int i = tid; i < D::G * D::TILES * 64; i += D::THREADS) sums[i] = 0.0;
    __syncthreads();

    float acc[64];
#pragma unroll
    for (int i = 0; i < 64; ++i) acc[i] = 0.0f;

    const int64_t nslabs = (d + D::TK - 1) / D::TK;
    const int64_t first = bx, step = gx;
    const int64_t mine = first < nslabs ? (nslabs - first + step - 1) / step : 0;

    auto flush = [&]() {
        reduce_scatter<64, 16>(acc, lane);               // 4 totals per lane
        const int b = scatter_base<64, 16>(lane);
        if (active) {
#pragma unroll
            for (int i = 0; i < 4; ++i) my_sums[b + i] += double(acc[i]);
        }
#pragma unroll
        for (int i = 0; i < 64; ++i) acc[i] = 0.0f;
    };

    if constexpr (VEC) {
        for (int s = 0; s < NSTAGE - 1; ++s) {
            if (s < mine) stage_slab<NB, true, ES>(stage + size_t(s) * D::R * D::TK, g, n, d, ld, (first + s * step) * D::TK);
            cp_async_commit();
        }
    }

    int since_flush = 0;
    for (int64_t it = 0; it < mine; ++it) {
        const float* cur;
        if constexpr (VEC) {
            cp_async_wait<NSTAGE - 2>();
            __syncthreads();
            const int64_t nxt = it + NSTAGE - 1;
            if (nxt < mine)
                stage_slab<NB, true, ES>(stage + size_t(nxt % NSTAGE) * D::R * D::TK, g, n, d, ld, (first + nxt * step) * D::TK);
            cp_async_commit();
            cur = stage + size_t(it % NSTAGE) * D::R * D::TK;
        } else {
            __syncthreads();
            stage_slab<NB, false>(stage, g, n, d, ld, (first + it * step) * D::TK, dtype);
            __syncthreads();
            cur = stage;
        }
        const int pa = grp * D::GQ + (I * 8) * D::TK4 + c, pb = grp * D::GQ + (J * 8) * D::TK4 + c;   // in units of four columns
        if (off_warp) {
#pragma unroll 1
            for (int k = 0; k < D::KQ; ++k) {          // rolled: the body is ~530 instructions already
                float4 a[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) a[i] = tile_ld4<ES>(cur, pa + i * D::TK4 + k * 16, dtype);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float4 b = tile_ld4<ES>(cur, pb + j * D::TK4 + k * 16, dtype);
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const float dx = a[i].x - b.x, dy = a[i].y - b.y, dz = a[i].z - b.z, dw = a[i].w - b.w;
                        float t = acc[i * 8 + j];
                        t = fmaf(dx, dx, t); t = fmaf(dy, dy, t); t = fmaf(dz, dz, t); t = fmaf(dw, dw, t);
                        acc[i * 8 + j] = t;
                    }
                }
            }
        } else {
            // two diagonal tiles: pairs i < j of tile I at acc[i*8+j], of tile J at acc[j*8+i]
#pragma unroll 1
            for (int k = 0; k < D::KQ; ++k) {
                float4 a[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) a[i] = tile_ld4<ES>(cur, pa + i * D::TK4 + k * 16, dtype);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
#pragma unroll
                    for (int j = i + 1; j < 8; ++j) {
                        const float dx = a[i].x - a[j].x, dy = a[i].y - a[j].y, dz = a[i].z - a[j].z, dw = a[i].w - a[j].w;
                        float t = acc[i * 8 + j];
                        t = fmaf(dx, dx, t); t = fmaf(dy, dy, t); t = fmaf(dz, dz, t); t = fmaf(dw, dw, t);
                        acc[i * 8 + j] = t;
                    }
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) a[i] = tile_ld4<ES>(cur, pb + i * D::TK4 + k * 16, dtype);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
#pragma unroll
                    for (int j = i + 1; j < 8; ++j) {
                        const float dx = a[i].x - a[j].x, dy = a[i].y - a[j].y, dz = a[i].z - a[j].z, dw = a[i].w - a[j].w;
                        float t = acc[j * 8 + i];
                        t = fmaf(dx, dx, t); t = fmaf(dy, dy, t); t = fmaf(dz, dz, t); t = fmaf(dw, dw, t);
                        acc[j * 8 + i] = t;
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
    double* my_partial = partials + size_t(bx) * kPairSlots;
    for (int i = tid; i < D::TILES * 64; i += D::THREADS) {
        double s = 0.0;
#pragma unroll 1
        for (int gq = 0; gq < D::G; ++gq) s += sums[size_t(gq) * D::TILES * 64 + i];
        my_partial[i] = s;
    }
    if (!last_cta_ticket(ticket, gx)) return;
    reduce_partials(partials, D::TILES * 64, D::THREADS, gx, [&](int i, double s) {
        const int t = i >> 6, hi = (i & 63) >> 3, lo = i & 7;
        int ra, rb;
        if (t < D::OFFJ) {
            int bi, bj;
            off_tile_blocks(t, NB, bi, bj);
            ra = bi * 8 + hi;
            rb = bj * 8 + lo;
        } else if (hi < lo) {                      // first diagonal tile of the job
            ra = 2 * (t - D::OFFJ) * 8 + hi;
            rb = 2 * (t - D::OFFJ) * 8 + lo;
        } else if (hi > lo && 2 * (t - D::OFFJ) + 1 < NB) {   // second one
            ra = (2 * (t - D::OFFJ) + 1) * 8 + lo;
            rb = (2 * (t - D::OFFJ) + 1) * 8 + hi;
        } else {
            ra = rb = n;                           // unused slot
        }
        if (ra < n && rb < n && ra < rb) {
            dist[ra * n + rb] = s;
            dist[rb * n + ra] = s;
        }
    });
    for (int i = tid; i < n; i += D::THREADS) dist[i * n + i] = 0.0;
    if (tid == 0) {
        *ticket = 0u;                           // ready for the next call
        if (path_word != nullptr) *path_word = kPathDifference;
    }
}

template <int NB, bool VEC, int ES = 4>
__global__ void __launch_bounds__(K1Dims<NB>::THREADS, K1Dims<NB>::MIN_CTAS)
k1_tiled(const float* __restrict__ g, int n, int64_t d, int64_t ld, double* __restrict__ dist,
         double* __restrict__ partials, unsigned int* __restrict__ ticket, unsigned int* __restrict__ path_word,
         const unsigned int* __restrict__ gate, int dtype) {
    // launched behind the tensor-core kernel, this one only runs if that kernel rejected its own
    // result (the gate word is written before this grid starts: same stream); the path word is
    // then that kernel's to write
    if (gate != nullptr && *gate == 0u) return;
    k1_tiled_body<NB, VEC, ES>(g, n, d, ld, dist, partials, ticket, gate == nullptr ? path_word : nullptr, dtype, blockIdx.x, gridDim.x);
}
// Batch mode: CTA b works on the tensor of descriptor multi[cta_desc[b]] (16-bit gradients: the
// element-by-element staging, VEC = false, only).
template <int NB, bool VEC>
__global__ void __launch_bounds__(K1Dims<NB>::THREADS, K1Dims<NB>::MIN_CTAS)
k1_tiled_multi(const MultiDesc* __restrict__ multi, const int* __restrict__ cta_desc, int n, double* __restrict__ dist,
               double* __restrict__ partials, unsigned int* __restrict__ tickets, int dtype) {
    const MultiDesc t = multi[cta_desc[blockIdx.x]];
    k1_tiled_body<NB, VEC, 4>(static_cast<const float*>(t.grads), n, t.d, t.ld, dist + size_t(t.index) * n * n,
                              partials + size_t(t.cta_first) * kPairSlots, tickets + t.index, nullptr, dtype,
                              blockIdx.x - unsigned(t.cta_first), unsigned(t.ctas));
}

// ------------------------------------------------------------------ launchers
template <typename K>
cudaError_t persistent_grid(K kern, int threads, size_t smem, int sm_count, int* per_sm_cache, int64_t work_items,
                            int64_t* grid_out) {
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    int per_sm = (dev >= 0 && dev < 64) ? per_sm_cache[dev] : 0;
    if (per_sm == 0) {
        if (smem > 48 * 1024) {
            err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
            if (err != cudaSuccess) return err;
        }
        if (smem > 0) {   // let several CTAs of shared memory fit on an SM
            err = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout,
                                       cudaSharedmemCarveoutMaxShared);
            if (err != cudaSuccess) return err;
        }
        err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, threads, smem);
        if (err != cudaSuccess) return err;
        if (per_sm < 1) per_sm = 1;
        if (dev >= 0 && dev < 64) per_sm_cache[dev] = per_sm;
    }
    int64_t grid = int64_t(sm_count) * per_sm;
    if (grid > kMaxCtasK1) grid = kMaxCtasK1;
    if (grid > work_items) grid = work_items;
    if (grid < 1) grid = 1;
    *grid_out = grid;
    return cudaSuccess;
}

template <int NB, bool VEC, int ES = 4>
cudaError_t launch_tiled(const float* g, int n, int64_t d, int64_t ld, double* dist, const Workspace& ws,
                         int sm_count, bool gated, cudaStream_t stream, int dtype = GAR_F32) {
    using D = K1Dims<NB>;
    static int per_sm_cache[64] = {0};
    int64_t grid = 1;
    cudaError_t err = persistent_grid(k1_tiled<NB, VEC, ES>, D::THREADS, D::SMEM_BYTES, sm_count, per_sm_cache,
                                      (d + D::TK - 1) / D::TK, &grid);
    if (err != cudaSuccess) return err;
    k1_tiled<NB, VEC, ES><<<unsigned(grid), D::THREADS, D::SMEM_BYTES, stream>>>(g, n, d, ld, dist, ws.partials(), ws.ticket(),
                                                                          ws.k1_path(), gated ? ws.k1_gate() : nullptr, dtype);
    return cudaGetLastError();
}

// A batch of tensors (fp32): one CTA per entry of cta_desc.
template <int NB, bool VEC>
cudaError_t launch_tiled_multi(const MultiDesc* desc, const int* cta_desc, int total_ctas, int n, double* dist, double* partials,
                               unsigned int* tickets, int dtype, cudaStream_t stream) {
    using D = K1Dims<NB>;
    static bool configured[64] = {false};
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (!(dev >= 0 && dev < 64 && configured[dev])) {
        err = cudaFuncSetAttribute(k1_tiled_multi<NB, VEC>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(D::SMEM_BYTES));
        if (err != cudaSuccess) return err;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    k1_tiled_multi<NB, VEC><<<unsigned(total_ctas), D::THREADS, D::SMEM_BYTES, stream>>>(desc, cta_desc, n, dist, partials, tickets, dtype);
    return cudaGetLastError();
}

template <int N, int V>
cudaError_t launch_direct(const float* g, int64_t d, int64_t ld, double* dist, const Workspace& ws, int sm_count,
                          cudaStream_t stream) {
    static int per_sm_cache[64] = {0};
    int64_t grid = 1;
    const int64_t nvec = d / V > 0 ? d / V : 1;
    constexpr size_t smem = K1RDims<N, V>::RING_BYTES;
    cudaError_t err = persistent_grid(k1_direct<N, V>, K1R_THREADS, smem, sm_count, per_sm_cache,
                                      (nvec + K1R_THREADS - 1) / K1R_THREADS, &grid);
    if (err != cudaSuccess) return err;
    k1_direct<N, V><<<unsigned(grid), K1R_THREADS, smem, stream>>>(g, d, ld, dist, ws.partials(), ws.ticket(), ws.k1_path());
    return cudaGetLastError();
}

// A batch of tensors through the ring kernel: one CTA per entry of cta_desc.
template <int N, int V>
cudaError_t launch_direct_multi(const MultiDesc* desc, const int* cta_desc, int total_ctas, double* dist, double* partials,
                                unsigned int* tickets, cudaStream_t stream) {
    constexpr size_t smem = K1RDims<N, V>::RING_BYTES;
    static bool configured[64] = {false};
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (!(dev >= 0 && dev < 64 && configured[dev])) {
        if (smem > 48 * 1024) {
            err = cudaFuncSetAttribute(k1_direct_multi<N, V>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
            if (err != cudaSuccess) return err;
        }
        err = cudaFuncSetAttribute(k1_direct_multi<N, V>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        if (err != cudaSuccess) return err;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    k1_direct_multi<N, V><<<unsigned(total_ctas), K1R_THREADS, smem, stream>>>(desc, cta_desc, dist, partials, tickets);
    return cudaGetLastError();
}
template <int N>
cudaError_t launch_direct_multi_n(const MultiDesc* desc, const int* cta_desc, int total_ctas, int vec, double* dist,
                                  double* partials, unsigned int* tickets, cudaStream_t stream) {
    if constexpr (N <= 8) {
        if (vec >= 4) return launch_direct_multi<N, 4>(desc, cta_desc, total_ctas, dist, partials, tickets, stream);
    }
    if (vec >= 2) return launch_direct_multi<N, 2>(desc, cta_desc, total_ctas, dist, partials, tickets, stream);
    return launch_direct_multi<N, 1>(desc, cta_desc, total_ctas, dist, partials, tickets, stream);
}

template <int N>
cudaError_t launch_direct_bulk(const void* g, int dtype, int64_t d, int64_t ld, double* dist, const Workspace& ws, int sm_count,
                               cudaStream_t stream) {
    static int per_sm_cache[64] = {0};
    using S = K1BShape<N>;
    const size_t smem = size_t(S::STAGES) * S::STAGE_BYTES;          // sized for fp32 rows; 16-bit rows use half of it
    int64_t grid = 0;
    cudaError_t err = persistent_grid(k1_direct_bulk<N>, S::THREADS, smem, sm_count, per_sm_cache, d / S::TC, &grid);
    if (err != cudaSuccess) return err;
    k1_direct_bulk<N><<<unsigned(grid), S::THREADS, smem, stream>>>(g, dtype, d, ld, dist, ws.partials(), ws.ticket(), ws.k1_error(),
                                                                     ws.k1_path());
    return cudaGetLastError();
}

// A batch of long tensors with 16-byte aligned rows through the staged kernel: one CTA per entry of cta_desc.
template <int N>
cudaError_t launch_direct_bulk_multi(const MultiDesc* desc, const int* cta_desc, int total_ctas, double* dist, double* partials,
                                     unsigned int* tickets, unsigned int* error_word, int dtype, cudaStream_t stream) {
    using S = K1BShape<N>;
    const size_t smem = size_t(S::STAGES) * S::STAGE_BYTES;
    static bool configured[64] = {false};
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (!(dev >= 0 && dev < 64 && configured[dev])) {
        err = cudaFuncSetAttribute(k1_direct_bulk_multi<N>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
        if (err != cudaSuccess) return err;
        err = cudaFuncSetAttribute(k1_direct_bulk_multi<N>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        if (err != cudaSuccess) return err;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    k1_direct_bulk_multi<N><<<unsigned(total_ctas), S::THREADS, smem, stream>>>(desc, cta_desc, dist, partials, tickets, error_word, dtype);
    return cudaGetLastError();
}

template <int N>
cudaError_t launch_direct_n(const float* g, int64_t d, int64_t ld, double* dist, const Workspace& ws, int sm_count,
                            cudaStream_t stream, int vec) {
    // 16-byte aligned rows and enough whole tiles for every SM: rows staged by bulk copies
    if (vec >= 4 && d >= int64_t(sm_count) * K1B_MIN_TC)
        return launch_direct_bulk<N>(g, GAR_F32, d, ld, dist, ws, sm_count, stream);
    // few rows: wide vectors keep enough bytes in flight; many rows: narrow ones keep the registers in check
    if constexpr (N <= 8) {
        if (vec >= 4) return launch_direct<N, 4>(g, d, ld, dist, ws, sm_count, stream);
    }
    if (vec >= 2) return launch_direct<N, 2>(g, d, ld, dist, ws, sm_count, stream);
    return launch_direct<N, 1>(g, d, ld, dist, ws, sm_count, stream);
}

}  // namespace

cudaError_t launch_distances(const float* grads, int n, int64_t d, int64_t ld, double* dist,
                             const Workspace& ws, int sm_count, int mode, cudaStream_t stream) {
    const uintptr_t addr = reinterpret_cast<uintptr_t>(grads);
    int vec = 1;
    if (addr % 16 == 0 && ld % 4 == 0) vec = 4;
    else if (addr % 8 == 0 && ld % 2 == 0) vec = 2;
    if (n == 1) return cudaMemsetAsync(dist, 0, sizeof(double), stream);
#define GAR_K1_DIRECT(NV) case NV: return launch_direct_n<NV>(grads, d, ld, dist, ws, sm_count, stream, vec);
#define GAR_K1_TILED(NBV)                                                                                  \
    case NBV:                                                                                              \
        return vec == 4 ? launch_tiled<NBV, true>(grads, n, d, ld, dist, ws, sm_count, gated, stream)       \
                        : launch_tiled<NBV, false>(grads, n, d, ld, dist, ws, sm_count, gated, stream);
    if (n <= 16) {
        switch (n) {
            GAR_K1_DIRECT(2) GAR_K1_DIRECT(3) GAR_K1_DIRECT(4) GAR_K1_DIRECT(5) GAR_K1_DIRECT(6) GAR_K1_DIRECT(7)
            GAR_K1_DIRECT(8) GAR_K1_DIRECT(9) GAR_K1_DIRECT(10) GAR_K1_DIRECT(11) GAR_K1_DIRECT(12)
            GAR_K1_DIRECT(13) GAR_K1_DIRECT(14) GAR_K1_DIRECT(15) GAR_K1_DIRECT(16)
        }
    }
    // Many rows and a long dimension: exact integer Gram product of rounded rows on the tensor
    // cores (HBM-bound), followed by the difference-form kernel behind a gate that the first one
    // opens only if its own bound on the rounding's effect is too large for some pair.  Short
    // dimensions keep the FP32 difference form, whose per-term error does not rely on averaging.
    bool gated = false;
    if (n > 16 && vec == 4 && d >= kMmaMinDim && mode == GAR_DISTANCES_AUTO) {
        const cudaError_t err = launch_distances_umma(grads, n, d, ld, dist, ws, sm_count, stream);
        if (err != cudaSuccess) return err;
        gated = true;
    }
    switch ((n + 7) / 8) {
        GAR_K1_TILED(3) GAR_K1_TILED(4) GAR_K1_TILED(5) GAR_K1_TILED(6) GAR_K1_TILED(7) GAR_K1_TILED(8)
    }
#undef GAR_K1_DIRECT
#undef GAR_K1_TILED
    return cudaErrorInvalidValue;
}

cudaError_t launch_distances_multi(const MultiDesc* desc, const int* cta_desc, int total_ctas, int n, int vec, double* dist,
                                   double* partials, unsigned int* tickets, unsigned int* error_word, int dtype, cudaStream_t stream) {
#define GAR_K1_MULTI_DIRECT(NV)                                                                                                  \
    case NV:                                                                                                                     \
        return vec == kMultiStaged                                                                                               \
                   ? launch_direct_bulk_multi<NV>(desc, cta_desc, total_ctas, dist, partials, tickets, error_word, dtype, stream)  \
                   : launch_direct_multi_n<NV>(desc, cta_desc, total_ctas, vec, dist, partials, tickets, stream);
#define GAR_K1_MULTI(NBV)                                                                                                        \
    case NBV:                                                                                                                    \
        return (vec == 4 && dtype == GAR_F32)                                                                                    \
                   ? launch_tiled_multi<NBV, true>(desc, cta_desc, total_ctas, n, dist, partials, tickets, dtype, stream)          \
                   : launch_tiled_multi<NBV, false>(desc, cta_desc, total_ctas, n, dist, partials, tickets, dtype, stream);
    // up to 16 rows: the staged kernel (either element size) or, fp32, the ring kernel; 16-bit
    // gradients that the staged kernel cannot take go through the tiled kernel
    if (n <= 16 && (dtype == GAR_F32 || vec == kMultiStaged)) {
        switch (n) {
            GAR_K1_MULTI_DIRECT(2) GAR_K1_MULTI_DIRECT(3) GAR_K1_MULTI_DIRECT(4) GAR_K1_MULTI_DIRECT(5) GAR_K1_MULTI_DIRECT(6)
            GAR_K1_MULTI_DIRECT(7) GAR_K1_MULTI_DIRECT(8) GAR_K1_MULTI_DIRECT(9) GAR_K1_MULTI_DIRECT(10) GAR_K1_MULTI_DIRECT(11)
            GAR_K1_MULTI_DIRECT(12) GAR_K1_MULTI_DIRECT(13) GAR_K1_MULTI_DIRECT(14) GAR_K1_MULTI_DIRECT(15) GAR_K1_MULTI_DIRECT(16)
        }
    }
    switch ((n + 7) / 8) {
        GAR_K1_MULTI(1) GAR_K1_MULTI(2) GAR_K1_MULTI(3) GAR_K1_MULTI(4) GAR_K1_MULTI(5) GAR_K1_MULTI(6) GAR_K1_MULTI(7)
        GAR_K1_MULTI(8)
    }
#undef GAR_K1_MULTI
#undef GAR_K1_MULTI_DIRECT
    return cudaErrorInvalidValue;
}

// Coordinates that are worth a CTA of its own in a batched distance launch (a few passes of the
// kernel's loop), for tensors whose alignment class is `vec`.
int distances_multi_chunk(int n, int vec, int dtype) {
    if (n <= 16 && vec == kMultiStaged) return 4 * K1B_MIN_TC;
    if (n <= 16 && dtype == GAR_F32) {
        const int v = (vec >= 4 && n <= 8) ? 4 : (vec >= 2 ? 2 : 1);
        return K1R_THREADS * v * 8;
    }
    switch ((n + 7) / 8) {
        case 1: return 4 * K1Dims<1>::TK; case 2: return 4 * K1Dims<2>::TK;
        case 3: return 4 * K1Dims<3>::TK; case 4: return 4 * K1Dims<4>::TK; case 5: return 4 * K1Dims<5>::TK;
        case 6: return 4 * K1Dims<6>::TK; case 7: return 4 * K1Dims<7>::TK; default: return 4 * K1Dims<8>::TK;
    }
}

// 16-bit gradients (bfloat16 / binary16): the staged direct kernel for n <= 16 when the rows are
// 16-byte aligned and d is large; else the tiled kernel, staging the raw 16-bit slabs by 16-byte
// copies (aligned rows) or element by element (any alignment), any n <= 64.  The arithmetic is the fp32 difference form throughout.
cudaError_t launch_distances_16(const void* grads, int dtype, int n, int64_t d, int64_t ld, double* dist,
                                const Workspace& ws, int sm_count, cudaStream_t stream) {
    if (n == 1) return cudaMemsetAsync(dist, 0, sizeof(double), stream);
    const uintptr_t addr = reinterpret_cast<uintptr_t>(grads);
    if (n <= 16 && addr % 16 == 0 && ld % 8 == 0 && d >= int64_t(sm_count) * K1B_MIN_TC) {
#define GAR_K1_BULK16(NV) case NV: return launch_direct_bulk<NV>(grads, dtype, d, ld, dist, ws, sm_count, stream);
        switch (n) {
            GAR_K1_BULK16(2) GAR_K1_BULK16(3) GAR_K1_BULK16(4) GAR_K1_BULK16(5) GAR_K1_BULK16(6) GAR_K1_BULK16(7)
            GAR_K1_BULK16(8) GAR_K1_BULK16(9) GAR_K1_BULK16(10) GAR_K1_BULK16(11) GAR_K1_BULK16(12)
            GAR_K1_BULK16(13) GAR_K1_BULK16(14) GAR_K1_BULK16(15) GAR_K1_BULK16(16)
        }
#undef GAR_K1_BULK16
    }
    const float* g = static_cast<const float*>(grads);       // only ever read as 16-bit elements
    const bool vec16 = addr % 16 == 0 && ld % 8 == 0;         // rows staged raw by 16-byte copies, else element by element
    // many rows, a long dimension, aligned rows: the tensor-core kernel (its producers widen the
    // values before they quantise them), with the tiled kernel behind its gate as for fp32
    bool gated = false;
    if (n > 16 && vec16 && d >= kMmaMinDim) {
        const cudaError_t err = launch_distances_umma(g, n, d, ld, dist, ws, sm_count, stream, dtype);
        if (err != cudaSuccess) return err;
        gated = true;
    }
#define GAR_K1_TILED16(NBV)                                                                                        \
    case NBV:                                                                                                      \
        return vec16 ? launch_tiled<NBV, true, 2>(g, n, d, ld, dist, ws, sm_count, gated, stream, dtype)            \
                     : launch_tiled<NBV, false>(g, n, d, ld, dist, ws, sm_count, gated, stream, dtype);
    switch ((n + 7) / 8) {
        GAR_K1_TILED16(1) GAR_K1_TILED16(2) GAR_K1_TILED16(3) GAR_K1_TILED16(4) GAR_K1_TILED16(5) GAR_K1_TILED16(6)
        GAR_K1_TILED16(7) GAR_K1_TILED16(8)
    }
#undef GAR_K1_TILED16
    return cudaErrorInvalidValue;
}

}  // namespace gar

namespace gar {
// ------------------------------------------------------------------------------------------
// Distances without any allocation.
//
// Some callers of this library cannot allocate device memory at the moment they need the
// distances: an aggregation hook that runs inside another framework's memory pool or under a
// fixed memory budget, a process that has handed all of its HBM to other buffers, or a
// latency-critical server loop where a cudaMalloc (which may synchronise the device) is not
// acceptable.  For them the scratch of the distance kernels -- the ticket counter and the
// per-CTA partial sums -- lives in the file-scope array below instead of a workspace.
// Its size is fixed: kStaticScratchBytes (about 10.9 MB), enough for the largest grid the
// distance kernels ever use and n <= GAR_MAX_N; every GPU that loads the library holds it
// until the process exits.
constexpr size_t kStaticScratchBytes = kCtrlBytes + kPartialBytes;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

namespace {
struct StaticScratchState {
    bool  ready = false;
    char* ptr = nullptr;
    int   sm_count = 0;
};
StaticScratchState g_static_state[64];
std::mutex g_static_mutex;             // guards the once-per-device set-up below
}  // namespace

}  // namespace gar

extern "C" int gar_pairwise_distances_static(const float* grads, int n, int64_t d, int64_t ld, double* dist,
                                             void* stream) {
    if (!grads || !dist || n < 1 || d < 1) return GAR_ERR_INVALID_ARG;
    if (n > GAR_MAX_N) return GAR_ERR_UNSUPPORTED;       // the static scratch is sized for n <= 64
    if (ld == 0) ld = d;
    if (ld < d) return GAR_ERR_INVALID_ARG;
    int dev = 0;
    if (int rc = gar::cuda_status(cudaGetDevice(&dev))) return rc;
    if (dev < 0 || dev >= 64) return GAR_ERR_UNSUPPORTED;
    gar::StaticScratchState& st = gar::g_static_state[dev];
    std::unique_lock<std::mutex> lock(gar::g_static_mutex);
    if (!st.ready) {
        // Once per device, with that device current: in host code the array's name is only a
        // stand-in; the address the kernels need comes from the runtime.
        void* p = nullptr;
        if (int rc = gar::cuda_status(cudaGetSymbolAddress(&p, gar::g_static_scratch))) return rc;
        if (p == nullptr) return gar::cuda_status(cudaErrorInvalidSymbol);
        if (int rc = gar::cuda_status(cudaDeviceGetAttribute(&st.sm_count, cudaDevAttrMultiProcessorCount, dev))) return rc;
        st.ptr = static_cast<char*>(p);
        st.ready = true;
    }
    lock.unlock();
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // the array keeps the previous call's contents: the ticket counter must start at zero
    // (the partial sums are overwritten before they are read)
    if (int rc = gar::cuda_status(cudaMemsetAsync(st.ptr, 0, gar::kCtrlBytes, s))) return rc;
    gar::Workspace ws{st.ptr};
    return gar::cuda_status(gar::launch_distances(grads, n, d, ld, dist, ws, st.sm_count, GAR_DISTANCES_AUTO, s));
}
