// Pairwise squared l2 distances for 16 < n <= 64 and large d on the tensor cores,
// as an EXACT integer Gram product (Algorithm 1, multi-Krum: the neighbour
// distances; D_ij = N_i + N_j - 2 P_ij with P = G G^T).
//
// The difference-form kernel needs n(n-1) FP32 instructions per coordinate and
// is bound by the FP32 pipe at n >= 23 (about twice its HBM time at n = 39, five
// times at n = 51).  A floating-point Gram product would be cheap on the tensor
// cores but loses digits by cancellation and by inexact accumulation.  Integer
// tensor-core arithmetic has neither problem:
//   * every row is quantised to 23-bit signed fixed point, x ~ q * 2^(E-148),
//     with a per-row exponent E that only grows while the CTA streams its
//     columns (round to nearest even, unbiased; the quantisation error of a
//     coordinate is at most 2^-23 of the row's running maximum);
//   * q is split into three signed 8-bit limbs q = l1*2^16 + l2*2^8 + l3;
//   * all six limb products (L1 L1^T, L2 L1^T, L3 L1^T, L2 L2^T, L3 L2^T,
//     L3 L3^T; the other three are their transposes) are accumulated with
//     mma.sync.m16n8k32.s8 in int32 -- exactly, so sum_t q_i q_j is exact;
//   * int32 sums are converted to fp64 (exact powers of two as scales) every
//     K1M_FLUSH slabs, or earlier when a row's exponent has to grow.
// Exact accumulation means identical rows give bit-identical sums and D = 0
// exactly, and no shift row is needed against cancellation.
//
// The CTA is warp-specialised.  Eight producer warps own the rows (row r belongs to
// warp r % 8): per 128-column slab a producer copies one float4 per lane and row
// with cp.async (coalesced 512 B) into a ring of raw slabs in shared memory, two
// or three slabs ahead (a lane only ever reads back what it copied itself, so the
// ring needs no barrier), then reduces the row's
// maximum with redux.sync, grows the row's exponent if needed (a row has a single
// owner, so no agreement between warps is required), quantises, transposes the limb
// bytes with prmt and stores three row-major int8 limb tiles (row stride 36 words:
// conflict-free ldmatrix rows) into one of two buffers.  Eight consumer warps
// issue the MMAs: warp (r, half) owns row tile r (16 rows) and MT column tiles
// (8 columns each); tiles on or above the diagonal compute all six products, tiles
// below it the three non-symmetric ones.  The consumers hold up to 96 int32
// accumulators per thread: the two producer warpgroups give registers back and the
// two consumer warpgroups take them (setmaxnreg).  Producers and consumers meet only at
// named barriers (full / empty per buffer).
#include <cstdlib>

#include "gar_internal.cuh"

namespace gar {
namespace {

constexpr int K1M_THREADS = 512;
constexpr int K1M_PRODUCERS = 8;        // warps 0..7
constexpr int K1M_CONSUMERS = 8;        // warps 8..15
constexpr int K1M_SLAB = 128;           // columns per slab (one float4 per lane)
constexpr int K1M_STRIDE = 36;          // words per limb-tile row (32 + 4 padding: conflict-free ldmatrix rows)
constexpr int K1M_FLUSH = 32;           // slabs between int32 -> fp64 flushes (|sum| < 2^27)
constexpr int K1M_MIN_EXP = 21;         // smallest row exponent (keeps the scale a normal float)
constexpr int K1M_PRODUCER_REGS = 96;    // per thread after setmaxnreg: 256 x 96 + 256 x 160 = 64 K registers
constexpr int K1M_CONSUMER_REGS = 160;
constexpr int K1M_LAUNCH_REGS = 128;     // 64 K registers / 512 threads
constexpr int K1M_TRI = 2080;           // entries (i <= j) of a 64 x 64 matrix

// named barriers (0 is __syncthreads)
constexpr int BAR_FULL = 1;             // +buffer
constexpr int BAR_EMPTY = 3;            // +buffer
constexpr int BAR_CONS = 5;             // consumers only

// followed in shared memory by the raw ring: float4 [stages][rows][32 lanes]
struct K1MSmem {
    unsigned limb[2][3][64][K1M_STRIDE]; // [buffer][limb: 0 = l1 (most significant)][row][4 columns per word]
    double   px[64][64];                 // 2^32 L1L1^T + 2^16 L2L2^T + L3L3^T       (tiles on or above the diagonal)
    double   py[64][64];                 // 2^24 L2L1^T + 2^16 L3L1^T + 2^8 L3L2^T   (all entries)
    int      slab_exp[2][64];            // exponent E each row of the buffer was quantised with
    int      cons_exp[64];               // exponents of the consumers' running int32 sums
    int      grow[2];                    // some row of the buffer uses a larger exponent than before
    unsigned nonfinite_lo, nonfinite_hi;
};

__device__ __forceinline__ unsigned prmt(unsigned a, unsigned b, unsigned sel) {
    unsigned r;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
    return r;
}

__device__ __forceinline__ void mma_s8(int (&c)[4], const unsigned (&a)[4], const unsigned (&b)[2]) {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc, int src_bytes) {
    unsigned sa = static_cast<unsigned>(__cvta_generic_to_shared(smem_dst));
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(sa), "l"(gsrc), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}

template <int MT> struct K1MRing {
    static constexpr int STAGES = MT == 4 ? 3 : 4;
    static constexpr size_t BYTES = size_t(STAGES) * MT * 16 * 32 * sizeof(float4);
};

__device__ __forceinline__ void ldmatrix_x4(unsigned (&r)[4], unsigned smem_addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_addr));
}

// The aligned barrier, ldmatrix and mma forms need the whole warp at the instruction together:
// reconverge after any lane-dependent branch before a barrier.
__device__ __forceinline__ void bar_sync(int id, int count) {
    __syncwarp();
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}
__device__ __forceinline__ void bar_arrive(int id, int count) {
    __syncwarp();
    asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(count) : "memory");
}

__device__ __forceinline__ double pow2(int e) {      // 2^e as a double, -1022 <= e <= 1023
    return __hiloint2double((1023 + e) << 20, 0);
}

__device__ __forceinline__ int tri_slot(int i, int j) {   // i <= j < 64 -> 0 .. 2079
    return i * 64 - (i * (i - 1)) / 2 + (j - i);
}

template <int MT>
__global__ void __launch_bounds__(K1M_THREADS, 1)
k1_mma(const float* __restrict__ g, int n, int64_t d, int64_t ld, double* __restrict__ dist,
       double* __restrict__ partials, unsigned int* __restrict__ ticket) {
    constexpr int ROWS = MT * 16;                            // padded row count
    constexpr int JR = ROWS / K1M_PRODUCERS;                 // rows per producer warp
    constexpr int NST = K1MRing<MT>::STAGES;                 // raw ring depth
    extern __shared__ __align__(16) unsigned char smem_raw[];
    K1MSmem& sm = *reinterpret_cast<K1MSmem*>(smem_raw);
    float4* ring = reinterpret_cast<float4*>(smem_raw + sizeof(K1MSmem));   // [NST][ROWS][32]
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    for (int i = tid; i < 64 * 64; i += K1M_THREADS) (&sm.px[0][0])[i] = 0.0;
    for (int i = tid; i < 64 * 64; i += K1M_THREADS) (&sm.py[0][0])[i] = 0.0;
    for (int i = tid; i < 2 * 3 * 64 * K1M_STRIDE; i += K1M_THREADS) (&sm.limb[0][0][0][0])[i] = 0u;
    if (tid < 64) { sm.cons_exp[tid] = K1M_MIN_EXP; sm.slab_exp[0][tid] = K1M_MIN_EXP; sm.slab_exp[1][tid] = K1M_MIN_EXP; }
    if (tid == 0) { sm.nonfinite_lo = 0u; sm.nonfinite_hi = 0u; sm.grow[0] = 0; sm.grow[1] = 0; }
    __syncthreads();

    const int64_t nslabs = (d + K1M_SLAB - 1) / K1M_SLAB;
    const int64_t first = blockIdx.x, step = gridDim.x;
    const int64_t mine = first < nslabs ? (nslabs - first + step - 1) / step : 0;

    if (warp < K1M_PRODUCERS) {
        // ================================================================ producers
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(K1M_PRODUCER_REGS));
        int row_exp[JR];
#pragma unroll
        for (int jr = 0; jr < JR; ++jr) row_exp[jr] = K1M_MIN_EXP;
        const int wpos = lane;                         // this lane's word: columns 4*lane .. 4*lane+3 of the slab
        // cp.async of this lane's float4 of every owned row of a slab into ring stage st
        const float* rowp[JR];                         // this lane's first float4 of every owned row
#pragma unroll
        for (int jr = 0; jr < JR; ++jr) {
            const int row = warp + jr * K1M_PRODUCERS;
            rowp[jr] = g + int64_t(row < n ? row : 0) * ld + 4 * lane;
        }
        auto request = [&](int st, int64_t slab) {
            const int64_t t0 = slab * K1M_SLAB;
            const int64_t left = d - t0 - 4 * lane;
            const int bytes = left >= 4 ? 16 : (left > 0 ? int(left) * 4 : 0);
            float4* dst = ring + size_t(st) * ROWS * 32 + warp * 32 + lane;
#pragma unroll
            for (int jr = 0; jr < JR; ++jr) {
                const int row = warp + jr * K1M_PRODUCERS;
                if (row < n) cp_async16(dst + jr * K1M_PRODUCERS * 32, bytes ? rowp[jr] + t0 : g, bytes);
            }
        };
#pragma unroll
        for (int s0 = 0; s0 < NST - 1; ++s0) {
            if (s0 < mine) request(s0, first + s0 * step);
            cp_async_commit();
        }
        for (int64_t it = 0; it < mine; ++it) {
            const int buf = int(it & 1);
            const int st = int(it % NST);
            cp_async_wait<NST - 2>();                                     // this lane's copies of slab `it` have landed
            {
                const int64_t nx = it + NST - 1;
                if (nx < mine) request(int(nx % NST), first + nx * step);  // stage last read one iteration ago
                cp_async_commit();
            }
            if (it >= 2) bar_sync(BAR_EMPTY + buf, K1M_THREADS);          // consumers are done with this buffer
            // phase 1: all owned rows' values and slab maxima (independent chains)
            float4 v[JR];
            int ex[JR];
#pragma unroll
            for (int jr = 0; jr < JR; ++jr) {
                const int row = warp + jr * K1M_PRODUCERS;
                v[jr] = row < n ? ring[(size_t(st) * ROWS + row) * 32 + lane] : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int jr = 0; jr < JR; ++jr) {
                const float m = fmaxf(fmaxf(fabsf(v[jr].x), fabsf(v[jr].y)), fmaxf(fabsf(v[jr].z), fabsf(v[jr].w)));
                // x - x is 0 for finite x and NaN otherwise: one flag for "some value is Inf or NaN"
                const float nf = ((v[jr].x - v[jr].x) + (v[jr].y - v[jr].y)) + ((v[jr].z - v[jr].z) + (v[jr].w - v[jr].w));
                const unsigned mb = (nf != nf) ? 0x7f800000u : __float_as_uint(m);
                ex[jr] = int(__reduce_max_sync(0xffffffffu, mb) >> 23);
            }
            // phase 2: exponents (branch-free), then quantisation, limb split and stores stage by
            // stage over all owned rows, so that the rows' dependent chains overlap
            bool grew = false, any_bad = false;
            float scale[JR];
#pragma unroll
            for (int jr = 0; jr < JR; ++jr) {
                const bool bad = ex[jr] == 255;
                const bool up = !bad && ex[jr] > row_exp[jr];
                row_exp[jr] = up ? ex[jr] + 1 : row_exp[jr];               // one binade of headroom
                grew |= up;
                any_bad |= bad;
                scale[jr] = __uint_as_float(unsigned(275 - row_exp[jr]) << 23);   // 2^(148-E)
            }
            if (any_bad) {                                                   // rare: a row holds Inf or NaN
#pragma unroll
                for (int jr = 0; jr < JR; ++jr) {
                    const int row = warp + jr * K1M_PRODUCERS;
                    if (ex[jr] == 255) {
                        v[jr] = make_float4(0.f, 0.f, 0.f, 0.f);            // quantised as zeros, flagged
                        if (lane == 0 && row < n) {
                            if (row < 32) atomicOr(&sm.nonfinite_lo, 1u << row); else atomicOr(&sm.nonfinite_hi, 1u << (row - 32));
                        }
                    }
                }
            }
            unsigned w[JR][4];
#pragma unroll
            for (int jr = 0; jr < JR; ++jr) {
                // round to nearest integer through the 1.5 * 2^23 trick; the low three bytes of
                // (q + 0x808080), each xor 0x80, are the signed limbs l3, l2, l1
                w[jr][0] = __float_as_uint(fmaf(v[jr].x, scale[jr], 12582912.0f)) + (0x00808080u - 0x4B400000u);
                w[jr][1] = __float_as_uint(fmaf(v[jr].y, scale[jr], 12582912.0f)) + (0x00808080u - 0x4B400000u);
                w[jr][2] = __float_as_uint(fmaf(v[jr].z, scale[jr], 12582912.0f)) + (0x00808080u - 0x4B400000u);
                w[jr][3] = __float_as_uint(fmaf(v[jr].w, scale[jr], 12582912.0f)) + (0x00808080u - 0x4B400000u);
            }
#pragma unroll
            for (int jr = 0; jr < JR; ++jr) {
                const int row = warp + jr * K1M_PRODUCERS;                  // rows >= n hold zeros: harmless stores
                const unsigned p01 = prmt(w[jr][0], w[jr][1], 0x5140u), p23 = prmt(w[jr][2], w[jr][3], 0x5140u);
                const unsigned h01 = prmt(w[jr][0], w[jr][1], 0x0062u), h23 = prmt(w[jr][2], w[jr][3], 0x0062u);
                sm.limb[buf][2][row][wpos] = prmt(p01, p23, 0x5410u) ^ 0x80808080u;   // l3
                sm.limb[buf][1][row][wpos] = prmt(p01, p23, 0x7632u) ^ 0x80808080u;   // l2
                sm.limb[buf][0][row][wpos] = prmt(h01, h23, 0x5410u) ^ 0x80808080u;   // l1
                if (lane == 0) sm.slab_exp[buf][row] = row_exp[jr];
            }
            if (grew && lane == 0) sm.grow[buf] = 1;
            __threadfence_block();
            bar_arrive(BAR_FULL + buf, K1M_THREADS);
        }
        cp_async_wait<0>();
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(K1M_LAUNCH_REGS));   // waits for the consumers' release
    } else {
        // ================================================================ consumers
        const int cw = warp - K1M_PRODUCERS;                  // 0..7
        const int ctid = tid - K1M_PRODUCERS * 32;            // 0..255
        const bool mma_warp = cw < 2 * MT;
        constexpr unsigned kRoles = MT == 2 ? 0x00003210u : (MT == 3 ? 0x00243150u : 0x72645310u);
        const int role = int((kRoles >> (4 * cw)) & 15u);
        const int rt = role >> 1, half = role & 1;
        const int gq = lane >> 2, cq = lane & 3;
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(K1M_CONSUMER_REGS));
        int acc[MT][6][4];                                    // [column tile][11, 21, 31, 22, 32, 33][fragment]
#pragma unroll
        for (int a = 0; a < MT; ++a)
#pragma unroll
            for (int p = 0; p < 6; ++p)
#pragma unroll
                for (int k = 0; k < 4; ++k) acc[a][p][k] = 0;

        // int32 sums -> fp64 with the exponents they were accumulated under; then zero them
        auto flush = [&]() {
            if (mma_warp) {
#pragma unroll
                for (int a = 0; a < MT; ++a) {
                    const int ct = half * MT + a;
                    const bool upper = ct >= 2 * rt;
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const int i = rt * 16 + gq + ((k & 2) ? 8 : 0);
                        const int j = ct * 8 + cq * 2 + (k & 1);
                        const int e = sm.cons_exp[i] + sm.cons_exp[j] - 296;      // s_i s_j = 2^e
                        // exact: |sums| < 2^27, so every bracket fits a double's 53 bits
                        const double y = ((double(acc[a][1][k]) * 256.0 + double(acc[a][2][k])) * 256.0 + double(acc[a][4][k])) * pow2(e + 8);
                        sm.py[i][j] += y;
                        if (upper) {                                       // warp-uniform; entries below the diagonal of a
                            const double x = double(acc[a][0][k]) * pow2(e + 32) +   // diagonal tile are kept but never read
                                             (double(acc[a][3][k]) * 65536.0 + double(acc[a][5][k])) * pow2(e);
                            sm.px[i][j] += x;
                        }
#pragma unroll
                        for (int p = 0; p < 6; ++p) acc[a][p][k] = 0;
                    }
                }
            }
        };

        int since_flush = 0;
        for (int64_t it = 0; it < mine; ++it) {
            const int buf = int(it & 1);
            bar_sync(BAR_FULL + buf, K1M_THREADS);                         // the buffer's limb tiles are written
            const bool grow = sm.grow[buf] != 0;                           // uniform: the scales change
            if (grow || since_flush == K1M_FLUSH) {                        // the one flush site of the loop
                flush();
                since_flush = 0;
            }
            if (grow) {
                bar_sync(BAR_CONS, K1M_CONSUMERS * 32);
                if (ctid < 64) sm.cons_exp[ctid] = sm.slab_exp[buf][ctid];
                if (ctid == 0) sm.grow[buf] = 0;
                bar_sync(BAR_CONS, K1M_CONSUMERS * 32);
            }
            if (mma_warp) {
                // ldmatrix addresses: lane l supplies the 16-byte row (l % 8) of matrix l / 8.
                // A (16 rows x 32 bytes): matrices (rows 0-7, bytes 0-15), (rows 8-15, 0-15), (rows 0-7, 16-31),
                // (rows 8-15, 16-31) = a0..a3.  B for two column tiles: (tile, bytes 0-15), (tile, 16-31),
                // (tile+1, 0-15), (tile+1, 16-31) = b0, b1 of the first tile, b0, b1 of the second.
                const int lrow = lane & 7, lmat = lane >> 3;
                const unsigned a_off = unsigned(((rt * 16 + lrow + (lmat & 1) * 8) * K1M_STRIDE + (lmat >> 1) * 4) * 4);
                const unsigned b_off = unsigned((((half * MT + (lmat >> 1)) * 8 + lrow) * K1M_STRIDE + (lmat & 1) * 4) * 4);
                const unsigned tile0 = static_cast<unsigned>(__cvta_generic_to_shared(&sm.limb[buf][0][0][0]));
                constexpr unsigned LIMB_BYTES = 64 * K1M_STRIDE * 4;
#pragma unroll 1
                for (int ks = 0; ks < 4; ++ks) {
                    const unsigned kb = ks * 32;                              // 32 bytes of every row per k-step
                    unsigned af[3][4];
#pragma unroll
                    for (int l = 0; l < 3; ++l) ldmatrix_x4(af[l], tile0 + l * LIMB_BYTES + a_off + kb);
#pragma unroll
                    for (int a2 = 0; a2 < MT; a2 += 2) {
                        unsigned bf[3][4];                                    // [limb][b0, b1 of tile a2; b0, b1 of tile a2+1]
#pragma unroll
                        for (int l = 0; l < 3; ++l)
                            ldmatrix_x4(bf[l], tile0 + l * LIMB_BYTES + b_off + unsigned(a2 * 8 * K1M_STRIDE * 4) + kb);
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            const int a = a2 + h;
                            if (a < MT) {
                                const int ct = half * MT + a;
                                const unsigned (&b1)[2] = *reinterpret_cast<const unsigned (*)[2]>(&bf[0][2 * h]);
                                const unsigned (&b2)[2] = *reinterpret_cast<const unsigned (*)[2]>(&bf[1][2 * h]);
                                const unsigned (&b3)[2] = *reinterpret_cast<const unsigned (*)[2]>(&bf[2][2 * h]);
                                mma_s8(acc[a][1], af[1], b1);            // L2 L1^T
                                mma_s8(acc[a][2], af[2], b1);            // L3 L1^T
                                mma_s8(acc[a][4], af[2], b2);            // L3 L2^T
                                if (ct >= 2 * rt) {                      // on or above the diagonal (warp-uniform)
                                    mma_s8(acc[a][0], af[0], b1);        // L1 L1^T
                                    mma_s8(acc[a][3], af[1], b2);        // L2 L2^T
                                    mma_s8(acc[a][5], af[2], b3);        // L3 L3^T
                                }
                            }
                        }
                    }
                }
            }
            if (it + 2 < mine) bar_arrive(BAR_EMPTY + buf, K1M_THREADS);   // hand the buffer back
            ++since_flush;
        }
        flush();
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(K1M_LAUNCH_REGS));   // back to the launch allocation
    }
    __syncthreads();

    // CTA partial: P_ij = px_ij + (py_ij + py_ji) for i <= j (the same expression on the diagonal,
    // so identical rows give bit-identical P_ii, P_ij, P_jj); slots 2300/2301: non-finite row masks
    double* my_partial = partials + size_t(blockIdx.x) * kPairSlots;
    for (int idx = tid; idx < 64 * 64; idx += K1M_THREADS) {
        const int i = idx >> 6, j = idx & 63;
        if (i <= j) my_partial[tri_slot(i, j)] = sm.px[i][j] + (sm.py[i][j] + sm.py[j][i]);
    }
    if (tid == 0) { my_partial[2300] = double(sm.nonfinite_lo); my_partial[2301] = double(sm.nonfinite_hi); }

    __shared__ int is_last;
    __threadfence();
    __syncthreads();
    if (tid == 0) is_last = (atomicAdd(ticket, 1u) == gridDim.x - 1);
    __syncthreads();
    if (!is_last) return;
    __threadfence();

    // last CTA: add the partials in CTA order, then D_ij = P_ii + P_jj - 2 P_ij
    double* ptot = &sm.py[0][0];                 // reuse: 2080 totals
    for (int s = tid; s < K1M_TRI; s += K1M_THREADS) {
        double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
        unsigned b = 0;
        for (; b + 4 <= gridDim.x; b += 4) {
            s0 += __ldcg(partials + size_t(b) * kPairSlots + s);
            s1 += __ldcg(partials + size_t(b + 1) * kPairSlots + s);
            s2 += __ldcg(partials + size_t(b + 2) * kPairSlots + s);
            s3 += __ldcg(partials + size_t(b + 3) * kPairSlots + s);
        }
        for (; b < gridDim.x; ++b) s0 += __ldcg(partials + size_t(b) * kPairSlots + s);
        ptot[s] = (s0 + s1) + (s2 + s3);
    }
    if (tid == 0) {
        unsigned lo = 0u, hi = 0u;
        for (unsigned b = 0; b < gridDim.x; ++b) {
            lo |= unsigned(__ldcg(partials + size_t(b) * kPairSlots + 2300));
            hi |= unsigned(__ldcg(partials + size_t(b) * kPairSlots + 2301));
        }
        sm.nonfinite_lo = lo; sm.nonfinite_hi = hi;
    }
    __syncthreads();
    const unsigned long long bad = (static_cast<unsigned long long>(sm.nonfinite_hi) << 32) | sm.nonfinite_lo;
    for (int idx = tid; idx < n * n; idx += K1M_THREADS) {
        const int i = idx / n, j = idx - i * n;
        double v = 0.0;
        if (i != j) {
            const int lo = i < j ? i : j, hi = i < j ? j : i;
            v = ptot[tri_slot(lo, lo)] + ptot[tri_slot(hi, hi)] - 2.0 * ptot[tri_slot(lo, hi)];
            if (v < 0.0) v = 0.0;
            if (((bad >> i) | (bad >> j)) & 1ull) v = INFINITY;
        }
        dist[idx] = v;
    }
    if (tid == 0) *ticket = 0u;               // ready for the next call
}

template <int MT>
cudaError_t launch_mt(const float* g, int n, int64_t d, int64_t ld, double* dist, const Workspace& ws, int sm_count,
                      cudaStream_t stream) {
    static int per_sm_cache[64] = {0};
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    int per_sm = (dev >= 0 && dev < 64) ? per_sm_cache[dev] : 0;
    const size_t smem = sizeof(K1MSmem) + K1MRing<MT>::BYTES;
    if (per_sm == 0) {
        err = cudaFuncSetAttribute(k1_mma<MT>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
        if (err != cudaSuccess) return err;
        err = cudaFuncSetAttribute(k1_mma<MT>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        if (err != cudaSuccess) return err;
        err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k1_mma<MT>, K1M_THREADS, smem);
        if (err != cudaSuccess) return err;
        if (per_sm < 1) per_sm = 1;
        if (dev >= 0 && dev < 64) per_sm_cache[dev] = per_sm;
    }
    const int64_t nslabs = (d + K1M_SLAB - 1) / K1M_SLAB;
    int64_t grid = int64_t(sm_count) * per_sm;
    if (grid > kMaxCtasK1) grid = kMaxCtasK1;
    if (grid > nslabs) grid = nslabs;
    k1_mma<MT><<<unsigned(grid), K1M_THREADS, smem, stream>>>(g, n, d, ld, dist, ws.partials(), ws.ticket());
    return cudaGetLastError();
}

}  // namespace

// 16 < n <= 64, grads 16-byte aligned, ld % 4 == 0.
cudaError_t launch_distances_mma(const float* grads, int n, int64_t d, int64_t ld, double* dist, const Workspace& ws,
                                 int sm_count, cudaStream_t stream) {
    if (n <= 32) return launch_mt<2>(grads, n, d, ld, dist, ws, sm_count, stream);
    if (n <= 48) return launch_mt<3>(grads, n, d, ld, dist, ws, sm_count, stream);
    return launch_mt<4>(grads, n, d, ld, dist, ws, sm_count, stream);
}

}  // namespace gar
