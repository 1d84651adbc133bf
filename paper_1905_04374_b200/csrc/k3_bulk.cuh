// Coordinate phase (Algorithm 1, multi-Bulyan: Median, Argpartition, Average), staged through
// shared memory by bulk copies.
//
// A tile is TC consecutive coordinates of every gradient the phase reads (the winners, and for
// the pre-aggregating rules every gradient of some set: "staged rows").  One lane of a producer
// warp fetches a tile with one bulk copy per staged row (TC * 4 contiguous bytes each) into a
// ring of stages; a stage's mbarrier counts the bytes in.  The compute threads own V adjacent
// coordinates of the tile each (V = 4, 2, 1 as the slot count grows and registers get scarce): all values they need sit in shared memory at offsets that are fixed at compile
// time for the winners (staged row s = slot s), so no address arithmetic, no load instruction per
// gradient and no exposed global-memory latency is left in their loop.  Every gradient is read
// from global memory exactly once.
//
// Pre-aggregation (G^agr[s] = mean over the set of slot s) follows the selection kernel's
// summation plan (layout in gar.h), restated branch-free:
//     T_s = T_{s-1} + cw_s * e_s        cw_s = 1 for a chained winner, else 0      (T_-1 = sum of base rows)
//     a_s = (T_s + C[col_s]) / m_s
// The corrections C (sums over the "loose" gradients) are evaluated first, once per correction slot
// in slot order, into a private shared-memory column per thread; col_s names the latest one at or
// before slot s (column 0 holds zero).
#pragma once
#include "k3_coordinate.cuh"
#include "mbar.cuh"

namespace gar {

// Shape of a CTA that gives every compute thread V adjacent coordinates of a tile.
template <int V> struct KBShape {
    static constexpr int CT = V == 1 ? 256 : 128;       // compute threads
    static constexpr int TC = CT * V;                   // coordinates per tile
    static constexpr int THREADS = CT + 32;             // + the producer warp
    static constexpr int ROW_BYTES = TC * 4;            // one staged row of a tile (one bulk copy)
};
constexpr int KB_MAX_STAGES = 4;
constexpr int KB_BAR_COMPUTE = 1;             // named barrier of the compute warps

struct alignas(16) KBSlot {
    float cw;        // 1: the slot's winner joins the running sum here
    float im;        // 1 / |set|
    int   coff;      // byte offset of the slot's correction column
    int   pad;
};

struct KBPlan {
    unsigned long long full[KB_MAX_STAGES];   // bulk copies -> compute threads: the stage's bytes have landed
    unsigned long long empty[KB_MAX_STAGES];  // compute warps -> producer: the stage has been read
    KBSlot   slot[GAR_MAX_N];
    int64_t  roff[GAR_MAX_N];                 // staged row -> element offset of its gradient
    int      theta, beta, median_of_agr, lo_pads;
    int      even_mean, median_only;
    int      nrows, nbase, ncorr, nstages;
    int      cols_in_stage;                   // the correction columns reuse dead rows of the stage
    uint8_t  col_row[GAR_MAX_N + 1];          // correction column -> row that holds it
    uint8_t  corr_dst[GAR_MAX_N];             // row the j-th correction is written to
    int      error;
    int      loose_row[GAR_MAX_N];            // loose gradient -> staged row
    int      saved_col[GAR_MAX_SAVED];
    uint8_t  corr_src[GAR_MAX_N];             // row of the column the correction starts from
    uint8_t  corr_nadd[GAR_MAX_N];
};

// Dynamic shared memory: [staged-row indices of the plan's additions, 16-byte padded]
// [correction columns (ncorr + 1) x TC floats] [stages: nrows x TC floats each].
// V values of a staged row at `p`: fp32, or (H16) 16-bit elements widened to fp32.
template <int V, bool H16> __device__ __forceinline__ void read_row(const unsigned char* p, int dtype, float (&x)[V]) {
    if constexpr (!H16) {
        read_vec<V>(reinterpret_cast<const float*>(p), x);
    } else if constexpr (V == 1) {
        x[0] = widen16(*reinterpret_cast<const unsigned short*>(p), dtype);
    } else if constexpr (V == 2) {
        const unsigned u = *reinterpret_cast<const unsigned*>(p);
        x[0] = widen16(static_cast<unsigned short>(u & 0xffffu), dtype);
        x[1] = widen16(static_cast<unsigned short>(u >> 16), dtype);
    } else {
        const uint2 u = *reinterpret_cast<const uint2*>(p);
        x[0] = widen16(static_cast<unsigned short>(u.x & 0xffffu), dtype);
        x[1] = widen16(static_cast<unsigned short>(u.x >> 16), dtype);
        x[2] = widen16(static_cast<unsigned short>(u.y & 0xffffu), dtype);
        x[3] = widen16(static_cast<unsigned short>(u.y >> 16), dtype);
    }
}

// H16: the gradients are 16-bit (bfloat16 or binary16 by `dtype`); the rows are staged as they are
// (half the bytes per copy) and widened when read; the correction columns stay fp32 in an area of
// their own.
template <int P, bool EXACT, bool PREAGG, int V, bool H16>
__global__ void __launch_bounds__(KBShape<V>::THREADS)
k3_bulk(const float* __restrict__ g, int n, int theta_arg, int64_t ntiles, int64_t ld, gar_selection_t* __restrict__ sel,
        const K3Out out, int pool_bytes, int dtype) {
    constexpr int KB_TC = KBShape<V>::TC, KB_CT = KBShape<V>::CT, KB_THREADS = KBShape<V>::THREADS;
    constexpr int ES = H16 ? 2 : 4;                                  // bytes per gradient element
    constexpr int KB_ROW_BYTES = KB_TC * ES;                         // one staged row of a tile (one bulk copy)
    constexpr int KB_COL_BYTES = KB_TC * 4;                          // one correction column (fp32)
    __shared__ KBPlan plan;
    extern __shared__ __align__(128) unsigned char kb_dyn[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    {
        const int status = k3_check(sel, n, theta_arg, PREAGG);
        if (status != GAR_OK) {                   // nothing usable: the output says so
            for (int64_t i = blockIdx.x; i < ntiles; i += gridDim.x)
                for (int c = tid; c < KB_TC; c += KB_THREADS) k3_store_nan(out, i * KB_TC + c);
            if (blockIdx.x == 0 && tid == 0 && sel->status == GAR_OK) sel->status = status;
            return;
        }
    }
    const int theta = EXACT ? P : sel->theta;

    // ---- plan -----------------------------------------------------------------------------
    const int nbase = PREAGG ? sel->nbase : 0;
    const int nloose = PREAGG ? sel->nloose : 0;
    const int nadds = PREAGG ? sel->total_adds : 0;
    for (int s = tid; s < GAR_MAX_N; s += KB_THREADS) {
        KBSlot sl;
        sl.cw = 0.0f; sl.im = 0.0f; sl.coff = 0; sl.pad = 0;
        if (s < theta) {
            const int r = theta - 1 - s;
            plan.roff[s] = int64_t(sel->winners[r]) * ld;
            sl.cw = ((sel->chain_mask >> s) & 1ull) ? 1.0f : 0.0f;
            sl.im = 1.0f / float(sel->m[r]);
        }
        plan.slot[s] = sl;
    }
    for (int k = tid; k < nbase; k += KB_THREADS) plan.roff[theta + k] = int64_t(sel->base_rows[k]) * ld;
    for (int u = tid; u < nloose; u += KB_THREADS) {        // a loose gradient that is also a winner shares its row
        const int row = sel->loose_rows[u];
        int match = -1;
        for (int s = 0; s < theta; ++s)
            if (sel->winners[theta - 1 - s] == row) match = s;
        plan.loose_row[u] = match;
    }
    __syncthreads();
    if (tid == 0) {
        int nrows = theta + nbase;
        for (int u = 0; u < nloose; ++u) {
            if (plan.loose_row[u] < 0) {
                plan.roff[nrows] = int64_t(sel->loose_rows[u]) * ld;
                plan.loose_row[u] = nrows++;
            }
        }
        plan.nrows = nrows;
        plan.nbase = nbase;
        plan.theta = theta;
        plan.beta = sel->beta;
        plan.median_of_agr = sel->median_of_agr;
        plan.even_mean = sel->even_median == GAR_EVEN_MEDIAN_MEAN ? 1 : 0;
        plan.median_only = sel->rule == GAR_MEDIAN ? 1 : 0;
        plan.lo_pads = (P - 1) / 2 - (theta - 1) / 2;
        plan.error = 0;
        // Corrections: column 0 holds zero, column j + 1 the j-th sum that has to be formed (a slot
        // that adds loose gradients).  A slot that only restarts from zero, continues, or takes up
        // a saved sum just names the column that already holds its value.
        int ncorr = 0, col = 0;
        int slot_col[GAR_MAX_N], src_col[GAR_MAX_N];
        if (PREAGG) {
            for (int s = 0; s < theta; ++s) {
                if ((sel->corr_mask >> s) & 1ull) {
                    const int src = sel->slot_src[s];
                    const int from = src == GAR_SRC_ZERO ? 0 : (src == GAR_SRC_CONT ? col : plan.saved_col[src]);
                    const int nadd = sel->slot_nadd[s];
                    if (nadd == 0) {
                        col = from;
                    } else {
                        src_col[ncorr] = from;
                        plan.corr_nadd[ncorr] = uint8_t(nadd);
                        col = ++ncorr;
                    }
                    const int sv = sel->slot_save[s];
                    if (sv != GAR_SAVE_NONE) plan.saved_col[sv] = col;
                }
                slot_col[s] = col;
            }
        }
        plan.ncorr = ncorr;
        // Where the columns live.  Rows of a stage that are dead by the time the corrections are
        // formed can hold them: the base rows (already summed) and the winners' rows (already in
        // registers) that no loose gradient shares.  If there are enough of them the columns cost
        // no shared memory and the ring gets it; else they get an area of their own.
        int nfree = 0;
        if (PREAGG) {
            for (int k = 0; k < nbase && nfree <= ncorr; ++k) plan.col_row[nfree++] = uint8_t(theta + k);
            for (int s = 0; s < theta && nfree <= ncorr; ++s) {
                bool shared_row = false;
                for (int u = 0; u < nloose; ++u) shared_row |= plan.loose_row[u] == s;
                if (!shared_row) plan.col_row[nfree++] = uint8_t(s);
            }
        }
        const bool in_stage = PREAGG && !H16 && nfree >= ncorr + 1;
        plan.cols_in_stage = in_stage ? 1 : 0;
        if (!in_stage)
            for (int c = 0; c <= ncorr; ++c) plan.col_row[c] = uint8_t(c);
        for (int j = 0; j < ncorr; ++j) {
            plan.corr_src[j] = plan.col_row[src_col[j]];
            plan.corr_dst[j] = plan.col_row[j + 1];
        }
        if (PREAGG)
            for (int s = 0; s < theta; ++s) plan.slot[s].coff = int(plan.col_row[slot_col[s]]) * KB_COL_BYTES;
        const int fixed = ((nadds + 15) & ~15) + (in_stage ? 0 : (ncorr + 1) * KB_COL_BYTES);
        int nst = (pool_bytes - fixed) / (nrows * KB_ROW_BYTES);
        if (nst > KB_MAX_STAGES) nst = KB_MAX_STAGES;
        plan.nstages = nst;
        if (nst < 1) plan.error = 1;                   // cannot happen with the launcher's pool size
        for (int st = 0; st < KB_MAX_STAGES; ++st) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(kb_smem_u32(&plan.full[st])), "r"(1u) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(kb_smem_u32(&plan.empty[st])), "r"(unsigned(KB_CT / 32)) : "memory");
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    uint8_t* const add_row = kb_dyn;
    for (int k = tid; k < nadds; k += KB_THREADS) add_row[k] = uint8_t(plan.loose_row[sel->add_pos[k]]);
    const int ncorr = plan.ncorr, nrows = plan.nrows, nstages = plan.nstages;
    float* const ccol = reinterpret_cast<float*>(kb_dyn + ((nadds + 15) & ~15));
    const bool cols_in_stage = plan.cols_in_stage != 0;
    unsigned char* const stages = reinterpret_cast<unsigned char*>(ccol) + (cols_in_stage ? 0 : (ncorr + 1) * KB_COL_BYTES);
    const unsigned stage_bytes = unsigned(nrows) * KB_ROW_BYTES;
    if (!cols_in_stage)
        for (int c = tid; c < KB_TC; c += KB_THREADS) ccol[c] = 0.0f;
    __syncthreads();
    volatile int* error = &plan.error;

    const int64_t first = blockIdx.x, step = gridDim.x;
    const int64_t mine = first < ntiles ? (ntiles - first + step - 1) / step : 0;

    if (warp == KB_CT / 32) {
        // ================================================================ producer
        // every lane fetches the staged rows lane, lane + 32, ...: a tile's copies leave together
        if (!*error) {
            int st = 0;
            unsigned parity = 1;                     // the phase before the first one: the first nstages waits pass
            int64_t i = 0;
            for (; i < mine; ++i) {
                if (!__all_sync(0xffffffffu, kb_wait(kb_smem_u32(&plan.empty[st]), parity, error))) break;
                const unsigned bar = kb_smem_u32(&plan.full[st]);
                if (lane == 0)
                    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(stage_bytes) : "memory");
                __syncwarp();
                const unsigned char* src = reinterpret_cast<const unsigned char*>(g) + (first + i * step) * (KB_TC * ES);
                const unsigned dst = kb_smem_u32(stages) + unsigned(st) * stage_bytes;
                for (int r = lane; r < nrows; r += 32)
                    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                                 ::"r"(dst + unsigned(r) * KB_ROW_BYTES), "l"(src + plan.roff[r] * ES), "r"(unsigned(KB_ROW_BYTES)), "r"(bar) : "memory");
                if (++st == nstages) { st = 0; parity ^= 1u; }
            }
            // no copy may be in flight when the CTA leaves: wait (bounded) for the last tiles issued,
            // also when a wait above gave up
            for (int64_t j = i > nstages ? i - nstages : 0; j < i; ++j)
                kb_wait(kb_smem_u32(&plan.full[j % nstages]), unsigned(j / nstages) & 1u, error, true);
        }
    } else {
        // ================================================================ compute: V coordinates per thread
        const int beta = plan.beta;
        const float inv_beta = 1.0f / float(beta);
        const int lo_pads = EXACT ? 0 : plan.lo_pads;
        const bool med_agr = PREAGG && plan.median_of_agr != 0;
        const bool even_mean = plan.even_mean != 0, median_only = plan.median_only != 0;
        int st = 0;
        unsigned parity = 0;
        bool ok = !*error;
        for (int64_t i = 0; ok && i < mine; ++i) {
            // one warp polls the stage's barrier, the others sleep in a hardware barrier meanwhile
            if (warp == 0) kb_wait(kb_smem_u32(&plan.full[st]), parity, error);
            unsigned failed;                      // the same answer in every compute thread
            asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.b32 q, %1, 0;\n\tbar.red.or.pred p, %2, %3, q;\n\tselp.b32 %0, 1, 0, p;\n\t}"
                         : "=r"(failed) : "r"(*error), "r"(KB_BAR_COMPUTE), "r"(KB_CT) : "memory");
            if (failed) break;
            unsigned char* const svb = stages + size_t(st) * stage_bytes + tid * V * ES;     // this thread's entries of the staged rows
            float* const mycol = cols_in_stage ? reinterpret_cast<float*>(svb) : ccol + tid * V;   // ... and of the correction columns' rows
            float e[P][V], a[P][V];
#pragma unroll
            for (int s = 0; s < P; ++s) {
                if (s < theta) {
                    read_row<V, H16>(svb + s * KB_ROW_BYTES, dtype, e[s]);
                } else {
#pragma unroll
                    for (int v = 0; v < V; ++v) e[s][v] = 0.0f;
                }
            }
            if constexpr (PREAGG) {
                float T[V];
#pragma unroll
                for (int v = 0; v < V; ++v) T[v] = 0.0f;
                const unsigned char* bp = svb + theta * KB_ROW_BYTES;
                int k = 0;
                for (; k + 4 <= nbase; k += 4) {
                    float x0[V], x1[V], x2[V], x3[V];
                    read_row<V, H16>(bp, dtype, x0); read_row<V, H16>(bp + KB_ROW_BYTES, dtype, x1);
                    read_row<V, H16>(bp + 2 * KB_ROW_BYTES, dtype, x2); read_row<V, H16>(bp + 3 * KB_ROW_BYTES, dtype, x3);
#pragma unroll
                    for (int v = 0; v < V; ++v) { T[v] += x0[v]; T[v] += x1[v]; T[v] += x2[v]; T[v] += x3[v]; }
                    bp += 4 * KB_ROW_BYTES;
                }
                for (; k < nbase; ++k) {
                    float x0[V];
                    read_row<V, H16>(bp, dtype, x0);
#pragma unroll
                    for (int v = 0; v < V; ++v) T[v] += x0[v];
                    bp += KB_ROW_BYTES;
                }
                {                                        // column 0: zero (its row's value has been used)
                    float z[V];
#pragma unroll
                    for (int v = 0; v < V; ++v) z[v] = 0.0f;
                    store_vec<V>(mycol + int(plan.col_row[0]) * KB_TC, z);
                }
                int kadd = 0;
                for (int j = 0; j < ncorr; ++j) {
                    float C[V];
                    read_vec<V>(mycol + int(plan.corr_src[j]) * KB_TC, C);
                    const int kend = kadd + plan.corr_nadd[j];
                    for (; kadd < kend; ++kadd) {
                        float x[V];
                        read_row<V, H16>(svb + int(add_row[kadd]) * KB_ROW_BYTES, dtype, x);
#pragma unroll
                        for (int v = 0; v < V; ++v) C[v] += x[v];
                    }
                    store_vec<V>(mycol + int(plan.corr_dst[j]) * KB_TC, C);
                }
#pragma unroll
                for (int s = 0; s < P; ++s) {
                    const float4 sl = *reinterpret_cast<const float4*>(&plan.slot[s]);      // cw, im, coff
                    float c[V];
                    read_vec<V>(reinterpret_cast<const float*>(reinterpret_cast<const unsigned char*>(mycol) + __float_as_int(sl.z)), c);
#pragma unroll
                    for (int v = 0; v < V; ++v) {
                        T[v] = fmaf(e[s][v], sl.x, T[v]);
                        a[s][v] = (T[v] + c[v]) * sl.y;
                    }
                }
            } else {
#pragma unroll
                for (int s = 0; s < P; ++s) {
#pragma unroll
                    for (int v = 0; v < V; ++v) a[s][v] = e[s][v];
                }
            }
            // the stage's values are in registers (or folded into T and C): hand it back; what this
            // thread wrote there must be ordered before the bulk copies that will overwrite it
            if (cols_in_stage) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0)
                asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(kb_smem_u32(&plan.empty[st])) : "memory");
            float res[V];
            k3_finish<P, V>(e, a, theta, beta, inv_beta, lo_pads, med_agr, even_mean, median_only, res);
            k3_store<V>(out, (first + i * step) * KB_TC + tid * V, res);
            if (++st == nstages) { st = 0; parity ^= 1u; }
        }
    }
    __syncthreads();
    if (tid == 0 && plan.error) sel->status = GAR_ERR_TIMEOUT;
}

}  // namespace gar
