// Pairwise squared distances (the D_ij that the scores of Eq. 4 sum) for 16 < n <= 64 with the
// Gram matrix on the fifth-generation tensor cores: tcgen05.mma, kind::i8, accumulators in
// tensor memory.
//
// Arithmetic.  Every row keeps a running exponent E; a value x is rounded to the integer
// q = rint(x * 2^(148-E)), |q| <= 2^22 (a relative step of 2^-21 of the row's largest binade), and q is split into three signed bytes q = l1 * 2^16 + l2 * 2^8 + l3.  With the byte matrices L1, L2,
// L3 (rows x columns) the Gram matrix of the rounded rows is
//     sum_ab 2^(8(3-a)) 2^(8(3-b)) La Lb^T        (a, b = 1..3),
// int8 x int8 products summed exactly in int32.  The six products with a <= b are formed, kept as
//     px = 2^32 L1L1^T + 2^16 L2L2^T + L3L3^T      (symmetric)
//     pz = 2^24 L1L2^T + 2^16 L1L3^T + 2^8 L2L3^T
// so that P = px + pz + pz^T, and D_ij = P_ii + P_jj - 2 P_ij.  Identical rows give identical
// entries P_ii = P_ij = P_jj and a distance of exactly 0.
//
// One CTA per SM, persistent over slabs of 128 columns, four kinds of warps:
//   producers (3 rows each)  cp.async ring -> quantise -> byte tiles in shared memory, laid out as
//                            the K-major, unswizzled operand of tcgen05.mma: 16-byte chunks of a
//                            row, rows in groups of eight (128 bytes), chunk stride LBO
//   one MMA warp             per slab 4 k-steps from one lane.  n <= 40 ("packed" tile: limb matrices
//                            40 rows apart, 128 rows in all): ONE 128 x 128 instruction per k-step with
//                            the tile as both operands, all nine limb products at once, 128 tensor-memory
//                            columns per accumulator set.  Larger n ("wide" tile, limb matrices 64 rows
//                            apart): two instructions per k-step,
//                            [L1; L2] x [L1; L2; L3]^T (128 x 192) and [L3; *] x L3^T (128 x 64; the lower 64
//                            rows of the second A run on into the next chunk and their products are never read),
//                            int32 accumulators in one of two sets of 256 tensor-memory columns
//   four flush warps         when a row's exponent grows (or after 256 slabs) the MMA warp moves to
//                            the other set; these warps read the closed set (tcgen05.ld, one warp
//                            per 32 lanes), scale by the exponents it was built under and add it,
//                            in fp64, into the CTA's px / pz arrays in shared memory
// Hand-offs are mbarriers (producer -> MMA, tcgen05.commit -> producer / flush, flush -> MMA);
// every wait is bounded: a wait that gives up raises an error flag, all roles leave their loops,
// the distance matrix is filled with NaN and the control block's error word is set.
//
// The last CTA also bounds what the rounding of the rows can have done to every distance (from the
// coarsest grid each row was rounded to) and, if some pair's bound exceeds 1e-6 of its distance,
// opens the gate of the difference-form kernel that the host has queued behind this one.
#include "gar_internal.cuh"
#include "mbar.cuh"

namespace gar {
namespace {

constexpr int KU_SLAB = 128;                 // columns per slab (one float4 per lane and row)
constexpr int KU_JR = 3;                     // rows per producer warp
constexpr int KU_MAX_NBUF = 6;               // byte-tile buffers at most
constexpr int KU_SBO = 128;                  // bytes between groups of eight rows
constexpr int KU_PACK_ROWS = 40;             // packed layout: rows per limb matrix
// Two layouts of a byte tile.  Wide (any n <= 64): limb matrices 64 rows apart, [L1; L2; L3] in 192
// rows, two instructions per k-step (see the file comment).  Packed (n <= 40): limb matrices 40
// rows apart, [L1; L2; L3; 8 zero rows] in 128 rows, which is both operands of ONE 128 x 128
// instruction per k-step that forms all nine limb products at once: half the operand bytes read
// by the tensor core, under half its multiply-accumulates, smaller tiles (more of them in flight).
template <bool PACKED> struct KUShape {
    static constexpr int LIMB_ROWS = PACKED ? KU_PACK_ROWS : 64;          // tile rows between limb matrices
    static constexpr int TILE_ROWS = PACKED ? 128 : 192;
    static constexpr int LBO = TILE_ROWS * 16 + 16;     // bytes between 16-byte column chunks (+ padding: conflict-free stores)
    static constexpr int BUF_BYTES = 8 * LBO;           // one slab: 8 chunks of 16 columns
    static constexpr int SET_COLS = PACKED ? 128 : 256; // tensor-memory columns per accumulator set
    static constexpr int NBUF = PACKED ? 5 : 3;         // byte-tile buffers
    // fp64 sums of the CTA: packed, one 40 x 40 array per limb of the row operand; wide, px and pz (64 x 64)
    static constexpr int SUM_DOUBLES = PACKED ? 3 * KU_PACK_ROWS * KU_PACK_ROWS : 2 * 4096;
};
constexpr int KU_PERIOD = 256;               // slabs per accumulator set at most: |sum| <= 256 * 128 * 2^14 = 2^29
constexpr int KU_MIN_EXP = 21;               // smallest row exponent (keeps the scale a normal float)
constexpr int KU_FLUSH_WARPS = 4;            // warps 0..3: tensor-memory lanes 32 w .. 32 w + 31
constexpr int KU_MMA_WARP = 4;
constexpr int KU_FIRST_PRODUCER = 5;
constexpr int KU_BAR_FLUSH = 1;              // named barrier of the flush warps
constexpr int KU_TRI = 2080;
constexpr double kGramRelBound = 1e-6;      // largest accepted bound on a distance's relative rounding error

struct KUSmem {
    unsigned long long full[KU_MAX_NBUF];        // producers -> MMA warp: the buffer's tiles are written
    unsigned long long empty[KU_MAX_NBUF];       // tcgen05.commit -> producers: the MMAs that read the buffer are done
    unsigned long long accfull[2];           // tcgen05.commit -> flush warps: the set is closed and complete
    unsigned long long accfree[2];           // flush warps -> MMA warp: the set has been read
    unsigned long long desc[KU_MAX_NBUF][8];     // operand descriptors of a buffer's MMAs: k-step ks at [ks] (rows 0..) and [4 + ks] (rows 128..)
    unsigned tmem_base;
    int      error;
    int      grow[KU_MAX_NBUF];                  // some row of the buffer uses a larger exponent than before
    int      set_last[2];                    // the set is the CTA's last one
    int      slab_exp[KU_MAX_NBUF][64];          // exponent each row of the buffer was quantised with
    int      set_exp[2][64];                 // exponents of the rows while the set was accumulated
    unsigned nonfinite_lo, nonfinite_hi;
    int      is_last;
    int      final_exp[64];                  // exponent each row ended with in this CTA (they only grow)
    int      reject;                         // last CTA: some distance's rounding bound is too large
};

__device__ __forceinline__ unsigned smem_u32(const void* p) { return kb_smem_u32(p); }

__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(unsigned* smem_dst, unsigned ncols) {      // whole warp
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_dst)), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(unsigned taddr, unsigned ncols) {         // whole warp
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

// Shared-memory operand descriptor: K-major, no swizzle.  Bits [0,14) address / 16, [16,30) chunk
// stride / 16, [32,46) eight-row-group stride / 16, [46,48) = 1 (descriptor version), layout type 0.
__device__ __forceinline__ unsigned long long umma_desc(unsigned saddr, int lbo) {
    return static_cast<unsigned long long>((saddr >> 4) & 0x3fffu) |
           (static_cast<unsigned long long>(lbo >> 4) << 16) |
           (static_cast<unsigned long long>(KU_SBO >> 4) << 32) | (1ull << 46);
}
// Instruction descriptor, kind::i8: int32 accumulators (2 at bit 4), signed 8-bit A and B (1 at bits
// 7 and 10), both K-major (bits 15, 16 clear), N / 8 at bit 17, M / 16 at bit 24.
__host__ __device__ constexpr unsigned umma_idesc(int m, int n) {
    return (2u << 4) | (1u << 7) | (1u << 10) | (unsigned(n >> 3) << 17) | (unsigned(m >> 4) << 24);
}
__device__ __forceinline__ void umma_i8(unsigned d_tmem, unsigned long long adesc, unsigned long long bdesc, unsigned idesc,
                                        unsigned accumulate) {                            // one thread
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
                 ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(0u) : "memory");
}
__device__ __forceinline__ void umma_commit(unsigned long long* bar) {                    // one thread
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// this thread's lane of tensor memory, 8 consecutive columns
__device__ __forceinline__ void tmem_ld8(unsigned taddr, int (&r)[8]) {                   // whole warp
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ unsigned prmt(unsigned a, unsigned b, unsigned sel) {
    unsigned r;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
    return r;
}
// Rounds the four values times `scale` to integers q through the 1.5 * 2^23 trick; w = q + 0x808080,
// whose low three bytes, each xor 0x80, are the signed bytes l1, l2, l3 of q.  `outside` collects the
// bits in which a result's sign and exponent field differ from those of [2^23, 2^24).
__device__ __forceinline__ void quantise4(const float4& v, float scale, unsigned (&w)[4], unsigned& outside) {
    const unsigned u0 = __float_as_uint(fmaf(v.x, scale, 12582912.0f)), u1 = __float_as_uint(fmaf(v.y, scale, 12582912.0f));
    const unsigned u2 = __float_as_uint(fmaf(v.z, scale, 12582912.0f)), u3 = __float_as_uint(fmaf(v.w, scale, 12582912.0f));
    outside |= (u0 ^ 0x4B000000u) | (u1 ^ 0x4B000000u);
    outside |= (u2 ^ 0x4B000000u) | (u3 ^ 0x4B000000u);
    w[0] = u0 + (0x00808080u - 0x4B400000u);
    w[1] = u1 + (0x00808080u - 0x4B400000u);
    w[2] = u2 + (0x00808080u - 0x4B400000u);
    w[3] = u3 + (0x00808080u - 0x4B400000u);
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

__device__ __forceinline__ double pow2(int e) { return __hiloint2double((1023 + e) << 20, 0); }   // -1022 <= e <= 1023
__device__ __forceinline__ int tri_slot(int i, int j) { return i * 64 - (i * (i - 1)) / 2 + (j - i); }   // i <= j < 64

// Shared memory: KUSmem, the byte-tile buffers, px and pz (2 x 64 x 64 doubles, stored transposed:
// [j][i]), the raw ring float4 [NST][3 * producer warps][32].
// FULL: n is a multiple of KU_JR, every producer warp owns KU_JR real rows (no per-row tests).
// H16: the gradients are 16-bit (bfloat16 or binary16 by `dtype`): a lane fetches 8 bytes per row and
// slab instead of 16 and widens its four values before it quantises them; everything after is the same.
template <int NST, int MAXT, bool FULL, bool PACKED, bool H16>
__global__ void __launch_bounds__(MAXT, 1)
k1_umma(const float* __restrict__ g, int dtype, int n, int64_t d, int64_t ld, double* __restrict__ dist,
        double* __restrict__ partials, unsigned int* __restrict__ ticket,
        unsigned int* __restrict__ error_word, unsigned int* __restrict__ path_word,
        unsigned int* __restrict__ gate_word) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    KUSmem& sm = *reinterpret_cast<KUSmem*>(smem_raw);
    constexpr int HEAD = (int(sizeof(KUSmem)) + 127) & ~127;
    using S = KUShape<PACKED>;
    constexpr int KU_NBUF = S::NBUF, KU_LBO = S::LBO, KU_BUF_BYTES = S::BUF_BYTES, KU_SET_COLS = S::SET_COLS;
    unsigned char* limb = smem_raw + HEAD;                                     // [KU_NBUF][KU_BUF_BYTES]
    double* px_t = reinterpret_cast<double*>(limb + KU_NBUF * KU_BUF_BYTES);    // wide: [64][64], px_t[j * 64 + i] = px_ij
    double* pz_t = px_t + 4096;                                                 // packed: [3][40][40] from px_t on
    float4* ring = reinterpret_cast<float4*>(px_t + S::SUM_DOUBLES);            // [NST][3 pw][32]
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nthreads = blockDim.x;
    const int pw = (nthreads >> 5) - KU_FIRST_PRODUCER;                        // producer warps
    const int ring_rows = KU_JR * pw;
    volatile int* error = &sm.error;

    for (int i = tid; i < (KU_NBUF * KU_BUF_BYTES + S::SUM_DOUBLES * 8) / 4; i += nthreads) reinterpret_cast<unsigned*>(limb)[i] = 0u;
    if (tid < 64) {
#pragma unroll
        for (int b = 0; b < KU_NBUF; ++b) sm.slab_exp[b][tid] = KU_MIN_EXP;
        sm.set_exp[0][tid] = KU_MIN_EXP;
        sm.set_exp[1][tid] = KU_MIN_EXP;
        sm.final_exp[tid] = KU_MIN_EXP;
    }
    if (tid == 0) {
#pragma unroll
        for (int b = 0; b < KU_NBUF; ++b) {
            kb_init(&sm.full[b], unsigned(pw));
            kb_init(&sm.empty[b], 1u);
            sm.grow[b] = 0;
        }
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            kb_init(&sm.accfull[s], 1u);
            kb_init(&sm.accfree[s], unsigned(KU_FLUSH_WARPS));
            sm.set_last[s] = 0;
        }
        sm.error = 0; sm.nonfinite_lo = 0u; sm.nonfinite_hi = 0u; sm.is_last = 0;
        kb_fence_init();
    }
    // the MMA warp's loop is one dependent instruction stream per slab and sits on the kernel's
    // critical path: everything it can look up instead of compute is tabulated here
    if (tid < KU_NBUF * 8) {
        const int b = tid >> 3, ks = tid & 3, second = (tid >> 2) & 1;
        sm.desc[b][tid & 7] = umma_desc(smem_u32(limb) + unsigned(b) * KU_BUF_BYTES + unsigned(ks) * 2u * KU_LBO + (second ? 128u * 16u : 0u), KU_LBO);
    }
    if (warp == KU_MMA_WARP) tmem_alloc(&sm.tmem_base, 2 * KU_SET_COLS);
    fence_async_smem();                  // the zeroed tiles are read by the tensor core (async proxy)
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem_base = sm.tmem_base;

    const int64_t nslabs = (d + KU_SLAB - 1) / KU_SLAB;
    const int64_t first = blockIdx.x, step = gridDim.x;
    const int64_t mine = first < nslabs ? (nslabs - first + step - 1) / step : 0;

    if (warp >= KU_FIRST_PRODUCER) {
        // ================================================================ producers
        // All shared-memory addresses are 32-bit window offsets and every per-slab quantity is kept
        // incrementally: this loop's instruction count bounds the kernel.
        const int p = warp - KU_FIRST_PRODUCER;
        int row_exp[KU_JR];
        float scale[KU_JR];                            // 2^(148 - row_exp)
        int exp_stores = 0;                            // tile buffers that still lack the rows' current exponents
        constexpr int ES = H16 ? 2 : 4;                // bytes per gradient element
        const char* nextp[KU_JR];                      // this lane's four columns of the next slab to request
        bool valid[KU_JR];
        unsigned tile_off[KU_JR];                      // byte offset of (row, this lane's 4 columns) in a tile buffer
#pragma unroll
        for (int jr = 0; jr < KU_JR; ++jr) {
            const int row = p + jr * pw;
            valid[jr] = FULL || row < n;
            row_exp[jr] = KU_MIN_EXP;
            scale[jr] = __uint_as_float(unsigned(275 - KU_MIN_EXP) << 23);
            nextp[jr] = reinterpret_cast<const char*>(g) + (int64_t(valid[jr] ? row : 0) * ld + first * KU_SLAB + 4 * lane) * ES;
            tile_off[jr] = unsigned(lane >> 2) * KU_LBO + unsigned(lane & 3) * 4 + unsigned(row) * 16;
        }
        const int64_t advance = step * KU_SLAB * ES;                               // bytes between this CTA's slabs
        const unsigned stage_bytes = unsigned(ring_rows) * 512u, row_stride = unsigned(pw) * 512u;
        const unsigned my_ring = smem_u32(ring) + unsigned(p * 32 + lane) * 16u;   // (stage 0, row p, this lane)
        const unsigned limb_u32 = smem_u32(limb);
        // the last slab of the matrix may be ragged: bytes of this lane's float4 that exist there
        const int64_t last_left = d - (nslabs - 1) * KU_SLAB - 4 * lane;
        const int last_bytes = last_left >= 4 ? 4 * ES : (last_left > 0 ? int(last_left) * ES : 0);
        const int last_it = (first + (mine - 1) * step == nslabs - 1) ? int(mine - 1) : -1;   // this CTA's iteration of it
        auto request = [&](unsigned stage_off, int it_req) {
            const int bytes = it_req == last_it ? last_bytes : 4 * ES;
#pragma unroll
            for (int jr = 0; jr < KU_JR; ++jr) {
                if (valid[jr]) {
                    const char* src = bytes ? nextp[jr] : reinterpret_cast<const char*>(g);   // nothing is read when bytes == 0
                    if constexpr (H16)
                        asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;\n"
                                     ::"r"(my_ring + stage_off + unsigned(jr) * row_stride), "l"(src), "r"(bytes) : "memory");
                    else
                        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n"
                                     ::"r"(my_ring + stage_off + unsigned(jr) * row_stride), "l"(src), "r"(bytes) : "memory");
                    nextp[jr] += advance;
                }
            }
        };
        const int nmine = int(mine);
        unsigned req_off = 0;                           // stage of the next request
#pragma unroll
        for (int s0 = 0; s0 < NST - 1; ++s0) {
            if (s0 < nmine) request(req_off, s0);
            cp_async_commit();
            req_off += stage_bytes;
        }
        unsigned cur_off = 0, buf_off = 0;              // stage being read, tile buffer being written
        int buf = 0;
        unsigned empty_parity = 1;          // parity of the phase before the first one: the first KU_NBUF waits pass
        for (int it = 0; it < nmine; ++it) {
            cp_async_wait<NST - 2>();                                     // this lane's copies of slab `it` have landed
            if (it + NST - 1 < nmine) request(req_off, it + NST - 1);     // into the stage read one iteration ago
            cp_async_commit();
            req_off += stage_bytes;
            if (req_off == unsigned(NST) * stage_bytes) req_off = 0;
            float4 v[KU_JR];
#pragma unroll
            for (int jr = 0; jr < KU_JR; ++jr) {
                v[jr] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (valid[jr]) {
                    if constexpr (H16) {
                        unsigned lo, hi;
                        asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(lo), "=r"(hi)
                                     : "r"(my_ring + cur_off + unsigned(jr) * row_stride) : "memory");
                        v[jr] = make_float4(widen16(static_cast<unsigned short>(lo & 0xffffu), dtype), widen16(static_cast<unsigned short>(lo >> 16), dtype),
                                            widen16(static_cast<unsigned short>(hi & 0xffffu), dtype), widen16(static_cast<unsigned short>(hi >> 16), dtype));
                    } else {
                        asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                                     : "=f"(v[jr].x), "=f"(v[jr].y), "=f"(v[jr].z), "=f"(v[jr].w)
                                     : "r"(my_ring + cur_off + unsigned(jr) * row_stride) : "memory");
                    }
                }
            }
            cur_off += stage_bytes;
            if (cur_off == unsigned(NST) * stage_bytes) cur_off = 0;
            // Common case: quantise with the rows' current scales.  x * scale + 1.5 * 2^23 lies in
            // [2^23, 2^24) (exponent field 150) exactly when |x * scale| stays inside the 2^22 range
            // of the three bytes; any other exponent field (a larger value, Inf, NaN) sends the warp
            // to the path below, which finds the rows' new exponents.
            unsigned w[KU_JR][4];
            unsigned outside = 0u;
#pragma unroll
            for (int jr = 0; jr < KU_JR; ++jr) quantise4(v[jr], scale[jr], w[jr], outside);
            bool grew = false;
            if (__any_sync(0xffffffffu, outside >= 0x00800000u)) {
                int ex[KU_JR];
#pragma unroll
                for (int jr = 0; jr < KU_JR; ++jr) {
                    // largest |value| of the slab row; x * 0 is 0 for finite x and NaN otherwise, so the sum
                    // below is the maximum, or NaN (exponent field 255) when a value is Inf or NaN
                    const float m = fmaxf(fmaxf(fabsf(v[jr].x), fabsf(v[jr].y)), fmaxf(fabsf(v[jr].z), fabsf(v[jr].w)));
                    const float nf = fmaf(v[jr].x, 0.f, fmaf(v[jr].y, 0.f, fmaf(v[jr].z, 0.f, v[jr].w * 0.f)));
                    ex[jr] = int(__reduce_max_sync(0xffffffffu, __float_as_uint(m + nf)) >> 23);   // >= 255: not finite
                }
#pragma unroll
                for (int jr = 0; jr < KU_JR; ++jr) {
                    const bool bad = ex[jr] >= 255;
                    const bool up = !bad && ex[jr] > row_exp[jr];
                    if (up) row_exp[jr] = ex[jr] + 1;                            // one binade of headroom
                    grew |= up;
                    scale[jr] = __uint_as_float(unsigned(275 - row_exp[jr]) << 23);   // 2^(148-E)
                    if (bad) {                                                   // a row holds Inf or NaN:
                        v[jr] = make_float4(0.f, 0.f, 0.f, 0.f);                // quantised as zeros, flagged
                        const int row = p + jr * pw;
                        if (lane == 0 && valid[jr]) {
                            if (row < 32) atomicOr(&sm.nonfinite_lo, 1u << row); else atomicOr(&sm.nonfinite_hi, 1u << (row - 32));
                        }
                    }
                    unsigned unused = 0u;
                    quantise4(v[jr], scale[jr], w[jr], unused);
                }
                exp_stores = KU_NBUF;                // every tile buffer gets the new exponents once
            }
            // the MMAs that read this buffer three slabs ago are done
            if (!kb_wait_warp(kb_smem_u32(&sm.empty[buf]), empty_parity, error)) break;
#pragma unroll
            for (int jr = 0; jr < KU_JR; ++jr) {
                if (valid[jr]) {
                    const unsigned p01 = prmt(w[jr][0], w[jr][1], 0x5140u), p23 = prmt(w[jr][2], w[jr][3], 0x5140u);
                    const unsigned h01 = prmt(w[jr][0], w[jr][1], 0x0062u), h23 = prmt(w[jr][2], w[jr][3], 0x0062u);
                    const unsigned at = limb_u32 + buf_off + tile_off[jr];
                    asm volatile("st.shared.b32 [%0], %1;" ::"r"(at), "r"(prmt(h01, h23, 0x5410u) ^ 0x80808080u) : "memory");             // l1
                    asm volatile("st.shared.b32 [%0+%2], %1;" ::"r"(at), "r"(prmt(p01, p23, 0x7632u) ^ 0x80808080u), "n"(S::LIMB_ROWS * 16) : "memory");   // l2
                    asm volatile("st.shared.b32 [%0+%2], %1;" ::"r"(at), "r"(prmt(p01, p23, 0x5410u) ^ 0x80808080u), "n"(S::LIMB_ROWS * 32) : "memory");   // l3
                }
            }
            if (exp_stores > 0) {                    // warp-uniform
                --exp_stores;
                if (lane == 0) {
#pragma unroll
                    for (int jr = 0; jr < KU_JR; ++jr)
                        if (valid[jr]) sm.slab_exp[buf][p + jr * pw] = row_exp[jr];
                }
            }
            if (grew && lane == 0) sm.grow[buf] = 1;
            fence_async_smem();                      // generic-proxy stores -> visible to the tensor core's reads
            __syncwarp();
            if (lane == 0) kb_arrive(&sm.full[buf]);
            buf_off += KU_BUF_BYTES;
            if (++buf == KU_NBUF) { buf = 0; buf_off = 0; empty_parity ^= 1u; }
        }
        cp_async_wait<0>();
        if (lane == 0) {
#pragma unroll
            for (int jr = 0; jr < KU_JR; ++jr)
                if (valid[jr]) sm.final_exp[p + jr * pw] = row_exp[jr];
        }
    } else if (warp == KU_MMA_WARP) {
        // ================================================================ MMA issue
        constexpr unsigned IDESC_A = umma_idesc(128, 192), IDESC_B = umma_idesc(128, 64), IDESC_P = umma_idesc(128, 128);
        const unsigned limb_addr = smem_u32(limb);
        int set = 0, since = 0;
        int opened0 = 0, opened1 = 0;
        bool have_open = false, fresh = true;
        int buf = 0;
        unsigned full_parity = 0;
        for (int64_t it = 0; it < mine; ++it) {
            if (!kb_wait_warp(kb_smem_u32(&sm.full[buf]), full_parity, error)) break;
            tc_fence_after();
            const bool grow = *reinterpret_cast<volatile int*>(&sm.grow[buf]) != 0;
            if (!have_open || grow || since == KU_PERIOD) {
                if (have_open) {                                            // close the running set
                    __syncwarp();
                    if (lane == 0) umma_commit(&sm.accfull[set]);
                    set ^= 1;
                }
                const int opened = set ? opened1 : opened0;
                if (opened > 0 && !kb_wait_warp(kb_smem_u32(&sm.accfree[set]), unsigned(opened - 1) & 1u, error)) break;
                tc_fence_after();
                sm.set_exp[set][lane] = sm.slab_exp[buf][lane];
                sm.set_exp[set][lane + 32] = sm.slab_exp[buf][lane + 32];
                if (lane == 0) { sm.grow[buf] = 0; sm.set_last[set] = 0; }
                __threadfence_block();
                __syncwarp();
                if (set) ++opened1; else ++opened0;
                have_open = true; fresh = true; since = 0;
            }
            if (lane == 0) {
                const unsigned d1 = tmem_base + unsigned(set * KU_SET_COLS), d2 = d1 + 192u;
                const unsigned long long* dt = sm.desc[buf];
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    const unsigned long long t1 = dt[ks];         // rows 0..: L1, L2, L3
                    const unsigned acc = (fresh && ks == 0) ? 0u : 1u;
                    if constexpr (PACKED) {
                        umma_i8(d1, t1, t1, IDESC_P, acc);      // [L1; L2; L3; 0] x [L1; L2; L3; 0]^T
                    } else {
                        const unsigned long long t3 = dt[4 + ks]; // rows 128..: L3, then unread rows
                        umma_i8(d1, t1, t1, IDESC_A, acc);      // [L1; L2] x [L1; L2; L3]^T
                        umma_i8(d2, t3, t3, IDESC_B, acc);      // [L3; *] x L3^T
                    }
                }
                umma_commit(&sm.empty[buf]);                    // arrives when these MMAs have read the buffer
            }
            __syncwarp();
            fresh = false;
            ++since;
            if (++buf == KU_NBUF) { buf = 0; full_parity ^= 1u; }
        }
        __syncwarp();
        if (lane == 0) {
            if (have_open) {
                sm.set_last[set] = 1;
                __threadfence_block();
                umma_commit(&sm.accfull[set]);
            } else {
                sm.error = 1;                                   // nothing was opened: a wait gave up at once
            }
        }
    } else {
        // ================================================================ flush: tensor memory -> fp64
        const int q = warp;                                     // lanes 32 q .. 32 q + 31 of tensor memory
        const int L = q * 32 + lane;
        // wide: lanes 0..63 are the rows of L1, 64..127 those of L2; packed: 40 lanes per limb
        const int limb_a = PACKED ? L / KU_PACK_ROWS : L >> 6;
        const int i = PACKED ? L - limb_a * KU_PACK_ROWS : L & 63;
        const bool lower = L >= 64;                             // wide: rows of L2 (L1 otherwise)
        for (int k = 0;; ++k) {
            const int set = k & 1;
            // a set closes rarely: poll slowly; then agree over the four warps (they meet at named barriers below)
            const bool ok = kb_wait_warp(kb_smem_u32(&sm.accfull[set]), unsigned(k >> 1) & 1u, error, 0u);
            unsigned all_ok;
            asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.b32 q, %1, 0;\n\tbar.red.and.pred p, %2, %3, q;\n\tselp.b32 %0, 1, 0, p;\n\t}"
                         : "=r"(all_ok) : "r"(unsigned(ok)), "r"(KU_BAR_FLUSH), "r"(KU_FLUSH_WARPS * 32) : "memory");
            if (!all_ok) { if (lane == 0) sm.error = 1; break; }
            tc_fence_after();
            const int last = *reinterpret_cast<volatile int*>(&sm.set_last[set]);
            const int ei = sm.set_exp[set][i & 63] - 296;
            const unsigned tbase = tmem_base + (unsigned(q * 32) << 16) + unsigned(set * KU_SET_COLS);
            if constexpr (PACKED) {
                // lane (a, i) holds row i of limb a against all three limbs of every row j: its share of
                // P_ij is 2^(8(2-a)) (2^16 LaL1^T + 2^8 LaL2^T + LaL3^T)_ij, an integer below 2^47 (exact),
                // times the rows' scales; it goes to the array of limb a, which no other lane writes
                double* mine_p = px_t + limb_a * (KU_PACK_ROWS * KU_PACK_ROWS);
#pragma unroll 1
                for (int j0 = 0; j0 < n; j0 += 8) {
                    int r0[8], r1[8], r2[8];
                    tmem_ld8(tbase + unsigned(j0), r0);
                    tmem_ld8(tbase + unsigned(KU_PACK_ROWS + j0), r1);
                    tmem_ld8(tbase + unsigned(2 * KU_PACK_ROWS + j0), r2);
                    tmem_ld_wait();
#pragma unroll
                    for (int t = 0; t < 8; ++t) {
                        const int j = j0 + t;
                        if (limb_a < 3 && i < n && j < n) {
                            const int e = ei + sm.set_exp[set][j] + 8 * (2 - limb_a);
                            const double v = (double(r0[t]) * 65536.0 + double(r1[t]) * 256.0) + double(r2[t]);
                            mine_p[j * KU_PACK_ROWS + i] += v * pow2(e);
                        }
                    }
                }
            } else {
#pragma unroll 1
                for (int phase = 0; phase < 2; ++phase) {
                    if ((phase == 1) == lower) {                    // warp-uniform: L1 rows first, then L2 rows
#pragma unroll 1
                        for (int j0 = 0; j0 < n; j0 += 8) {
                            int r0[8], r1[8], r2[8], r3[8];
                            if (!lower) {
                                tmem_ld8(tbase + unsigned(j0), r0);             // L1 L1^T
                                tmem_ld8(tbase + unsigned(64 + j0), r1);        // L1 L2^T
                                tmem_ld8(tbase + unsigned(128 + j0), r2);       // L1 L3^T
                                tmem_ld8(tbase + unsigned(192 + j0), r3);       // L3 L3^T
                            } else {
                                tmem_ld8(tbase + unsigned(64 + j0), r0);        // L2 L2^T
                                tmem_ld8(tbase + unsigned(128 + j0), r1);       // L2 L3^T
#pragma unroll
                                for (int t = 0; t < 8; ++t) { r2[t] = 0; r3[t] = 0; }
                            }
                            tmem_ld_wait();
#pragma unroll
                            for (int t = 0; t < 8; ++t) {
                                const int j = j0 + t;
                                const int e = ei + sm.set_exp[set][j & 63];       // s_i s_j = 2^e
                                double x, y;                                      // exact: |sums| < 2^30
                                if (!lower) {
                                    x = double(r0[t]) * pow2(e + 32) + double(r3[t]) * pow2(e);
                                    y = (double(r1[t]) * 256.0 + double(r2[t])) * pow2(e + 16);
                                } else {
                                    x = double(r0[t]) * pow2(e + 16);
                                    y = double(r1[t]) * pow2(e + 8);
                                }
                                if (i < n && j < n) {
                                    px_t[j * 64 + i] += x;
                                    pz_t[j * 64 + i] += y;
                                }
                            }
                        }
                    }
                    asm volatile("bar.sync %0, %1;" ::"r"(KU_BAR_FLUSH), "r"(KU_FLUSH_WARPS * 32) : "memory");
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) kb_arrive(&sm.accfree[set]);
            if (last) break;
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == KU_MMA_WARP) tmem_dealloc(tmem_base, 2 * KU_SET_COLS);

    // CTA partial: P_ij = px_ij + (pz_ij + pz_ji) for i <= j (the same expression on the diagonal, so
    // identical rows give bit-identical P_ii, P_ij, P_jj); then the rows' final exponents, the
    // non-finite row masks and the error flag
    double* my_partial = partials + size_t(blockIdx.x) * kPairSlots;
    for (int idx = tid; idx < 64 * 64; idx += nthreads) {
        const int i = idx >> 6, j = idx & 63;
        if (i <= j) {
            double v = 0.0;
            if (j < n) {
                if constexpr (PACKED) {
                    constexpr int PP = KU_PACK_ROWS * KU_PACK_ROWS;
                    v = (px_t[j * KU_PACK_ROWS + i] + px_t[PP + j * KU_PACK_ROWS + i]) + px_t[2 * PP + j * KU_PACK_ROWS + i];
                } else {
                    v = px_t[j * 64 + i] + (pz_t[j * 64 + i] + pz_t[i * 64 + j]);
                }
            }
            my_partial[tri_slot(i, j)] = v;
        }
    }
    if (tid < 64) my_partial[kSlotRowExp + tid] = double(sm.final_exp[tid]);
    if (tid == 0) {
        my_partial[kSlotNonfinite] = double(sm.nonfinite_lo);
        my_partial[kSlotNonfinite + 1] = double(sm.nonfinite_hi);
        my_partial[kSlotError] = double(sm.error);
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) sm.is_last = (atomicAdd(ticket, 1u) == gridDim.x - 1);
    __syncthreads();
    if (!sm.is_last) return;
    __threadfence();

    // last CTA: add the partials in CTA order, then D_ij = P_ii + P_jj - 2 P_ij
    double* ptot = reinterpret_cast<double*>(limb);              // reuse: 2080 totals
    for (int s = tid; s < KU_TRI; s += nthreads) {
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
        unsigned lo = 0u, hi = 0u, err = 0u;
        for (unsigned b = 0; b < gridDim.x; ++b) {
            lo |= unsigned(__ldcg(partials + size_t(b) * kPairSlots + kSlotNonfinite));
            hi |= unsigned(__ldcg(partials + size_t(b) * kPairSlots + kSlotNonfinite + 1));
            err |= unsigned(__ldcg(partials + size_t(b) * kPairSlots + kSlotError));
        }
        sm.nonfinite_lo = lo; sm.nonfinite_hi = hi; sm.error = int(err);
        if (err) *error_word = 1u;
    }
    if (tid >= 64 && tid < 128) {                 // the coarsest grid any CTA used for each row
        int e = KU_MIN_EXP;
        for (unsigned b = 0; b < gridDim.x; ++b) e = max(e, int(__ldcg(partials + size_t(b) * kPairSlots + kSlotRowExp + (tid - 64))));
        sm.final_exp[tid - 64] = e;
    }
    __syncthreads();
    const unsigned long long bad = (static_cast<unsigned long long>(sm.nonfinite_hi) << 32) | sm.nonfinite_lo;
    const bool failed = sm.error != 0;
    // What the rounding of the rows can have done to a distance.  With steps s_i, s_j (the coarsest
    // each row saw) the rounding errors e_i, e_j of a coordinate lie within half a step:
    //   D'_ij - D_ij = sum (e_i - e_j)^2 + 2 sum (x_i - x_j)(e_i - e_j),
    // a bias of at most d (s_i^2 + s_j^2) / 12 on average and a zero-mean term of standard deviation
    // 2 sqrt(D_ij (s_i^2 + s_j^2) / 12) when the errors are independent of the differences; six
    // standard deviations are allowed for.  A pair whose bound exceeds 1e-6 of its distance rejects
    // the matrix (the caller's next kernel recomputes it from differences).  Rows that agree within
    // the grid everywhere give exactly 0 and are left at that.
    bool reject = false;
    for (int idx = tid; idx < n * n; idx += nthreads) {
        const int i = idx / n, j = idx - i * n;
        double v = 0.0;
        if (i != j) {
            const int lo = i < j ? i : j, hi = i < j ? j : i;
            v = ptot[tri_slot(lo, lo)] + ptot[tri_slot(hi, hi)] - 2.0 * ptot[tri_slot(lo, hi)];
            if (v < 0.0) v = 0.0;
            if (((bad >> i) | (bad >> j)) & 1ull) {
                v = INFINITY;
            } else if (v > 0.0) {
                const double m2 = pow2(2 * (sm.final_exp[i] - 148)) + pow2(2 * (sm.final_exp[j] - 148));
                const double bound = double(d) * m2 * (1.0 / 12.0) + 12.0 * sqrt(v * m2 * (1.0 / 12.0));
                reject |= bound > kGramRelBound * v;
            }
        }
        dist[idx] = failed ? __longlong_as_double(0x7ff8000000000000ll) : v;
    }
    const int any_reject = __syncthreads_or(reject ? 1 : 0);
    if (tid == 0) {
        const bool redo = any_reject && !failed;
        *gate_word = redo ? 1u : 0u;
        *path_word = redo ? kPathGramRejected : kPathGram;
        *ticket = 0u;                           // ready for the next call
    }
}

template <int NST, int MAXT, bool FULL, bool PACKED, bool H16>
cudaError_t launch_ku(const float* g, int dtype, int n, int64_t d, int64_t ld, double* dist, const Workspace& ws, int sm_count,
                      int pw, size_t smem, cudaStream_t stream) {
    static size_t configured[64] = {0};                        // dynamic shared memory the kernel is allowed, per device
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= 64 || configured[dev] < smem) {
        err = cudaFuncSetAttribute(k1_umma<NST, MAXT, FULL, PACKED, H16>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
        if (err != cudaSuccess) return err;
        if (dev >= 0 && dev < 64) configured[dev] = smem;
    }
    // one CTA per SM: every CTA owns all 512 tensor-memory columns of its SM (the shared memory it
    // asks for, more than half an SM's, keeps a second CTA away)
    const int64_t nslabs = (d + KU_SLAB - 1) / KU_SLAB;
    int64_t grid = sm_count;
    if (grid > kMaxCtasK1) grid = kMaxCtasK1;
    if (grid > nslabs) grid = nslabs;
    k1_umma<NST, MAXT, FULL, PACKED, H16><<<unsigned(grid), 32 * (KU_FIRST_PRODUCER + pw), smem, stream>>>(
        g, dtype, n, d, ld, dist, ws.partials(), ws.ticket(), ws.k1_error(), ws.k1_path(), ws.k1_gate());
    return cudaGetLastError();
}

}  // namespace

// 16 < n <= 64, grads 16-byte aligned, ld % 4 == 0.
template <bool PACKED, bool H16>
static cudaError_t launch_umma_layout(const float* grads, int dtype, int n, int64_t d, int64_t ld, double* dist, const Workspace& ws,
                                      int sm_count, cudaStream_t stream) {
    using S = KUShape<PACKED>;
    const int pw = (n + KU_JR - 1) / KU_JR;                    // producer warps: three rows each
    const size_t fixed = ((sizeof(KUSmem) + 127) & ~size_t(127)) + size_t(S::NBUF) * S::BUF_BYTES + size_t(S::SUM_DOUBLES) * sizeof(double);
    const size_t stage = size_t(KU_JR) * pw * 32 * sizeof(float4);
    constexpr size_t kSmemMax = 227 * 1024;                    // per-CTA limit of the SM
    constexpr int kSmall = 32 * (KU_FIRST_PRODUCER + 14), kLarge = 32 * (KU_FIRST_PRODUCER + 22);
    int nst = 4;
    while (nst > 2 && fixed + nst * stage > kSmemMax) --nst;   // deepest raw ring that fits
    const size_t smem = fixed + nst * stage;
#define GAR_KU(NSTV, MAXTV)                                                                                           \
    do {                                                                                                              \
        if (n == KU_JR * pw) return launch_ku<NSTV, MAXTV, true, PACKED, H16>(grads, dtype, n, d, ld, dist, ws, sm_count, pw, smem, stream); \
        return launch_ku<NSTV, MAXTV, false, PACKED, H16>(grads, dtype, n, d, ld, dist, ws, sm_count, pw, smem, stream);           \
    } while (0)
    if (pw <= 14) { if (nst == 4) GAR_KU(4, kSmall); if (nst == 3) GAR_KU(3, kSmall); GAR_KU(2, kSmall); }
    if constexpr (!PACKED) {
        if (nst == 4) GAR_KU(4, kLarge);
        if (nst == 3) GAR_KU(3, kLarge);
        GAR_KU(2, kLarge);
    }
#undef GAR_KU
    return cudaErrorInvalidValue;
}

cudaError_t launch_distances_umma(const float* grads, int n, int64_t d, int64_t ld, double* dist, const Workspace& ws,
                                  int sm_count, cudaStream_t stream, int dtype) {
    if (dtype == GAR_F32) {
        if (n <= KU_PACK_ROWS) return launch_umma_layout<true, false>(grads, dtype, n, d, ld, dist, ws, sm_count, stream);
        return launch_umma_layout<false, false>(grads, dtype, n, d, ld, dist, ws, sm_count, stream);
    }
    if (n <= KU_PACK_ROWS) return launch_umma_layout<true, true>(grads, dtype, n, d, ld, dist, ws, sm_count, stream);
    return launch_umma_layout<false, true>(grads, dtype, n, d, ld, dist, ws, sm_count, stream);
}

}  // namespace gar
