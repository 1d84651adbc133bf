// Scoring and iterative selection from the n x n distance matrix in one CTA
// (Eq. 4; Algorithm 1: function multi-Krum and the extraction loop of
// multi-Bulyan).  Nothing here touches the gradients: the distance matrix is
// reused by every round.
//
//  1. D is loaded into shared memory (non-finite entries become +inf).
//  2. Every row's distances to the other rows are sorted once, by counting,
//     on (value, index).
//  3. Round r (k = n-r gradients left): one warp per row walks the row's sorted
//     list, skips extracted gradients and adds the first q = k-f-2 values in
//     fp64 (fixed shuffle tree); rows are then ranked on (score, index); the
//     winner is rank 0 and the round's set the m best ranks; the winner is
//     removed.
//  4. The summation schedule of the coordinate phase is derived from the sets.
#include "gar_internal.cuh"

namespace gar {
namespace {

constexpr int K2_THREADS = 1024;
constexpr int NMAX = GAR_MAX_N;

struct K2Smem {
    double   dm[NMAX][NMAX];      // sanitised distances
    double   sv[NMAX][NMAX];      // per row: other rows' distances, ascending
    uint8_t  sj[NMAX][NMAX];      // per row: their indices
    double   score[NMAX];
    double   pick[NMAX][4];       // per round: s(1), s(2), s(m), s(m+1)
    uint8_t  order[NMAX][NMAX];   // per round: the remaining rows by rank (ranks are distinct: one writer per entry)
    unsigned long long alive;
};

__device__ __forceinline__ double rel_gap(double lo, double hi) {
    if (!isfinite(hi)) return isfinite(lo) ? INFINITY : 0.0;
    if (hi <= 0.0) return 0.0;
    return (hi - lo) / hi;
}

// Derive the coordinate kernel's summation plan from winners[] and sets[] (the
// layout is described in gar.h).  Slots are rounds in reverse (slot s = round
// theta-1-s).  Gradients present in every slot form the base; a winner that
// stays in every set from its own slot on is "chained" (added to the running sum
// at its slot); everything else is "loose" and summed per slot into a correction
// C_s by the cheapest of: start from zero, continue from slot s-1 (if that loose
// set is a subset) or start from a saved earlier C (if a subset).  Sums are only
// ever added to.  At most GAR_MAX_SAVED corrections are kept.
struct PlanSmem {
    unsigned long long slotset[NMAX];   // full set of slot s
    unsigned long long loose[NMAX];     // loose part of slot s
    unsigned long long addmask[NMAX];
    unsigned long long uni, base, chain, loose_all;
    int choice[NMAX];       // pass 1: chosen earlier slot (>= 0), -1 zero, -2 continue
    int usage[NMAX];
    int saved[NMAX];        // slot -> saved index or -1
    int offset[NMAX + 1];
    // shared-memory copies of what the single-threaded passes walk over (a dependent chain of
    // global loads per slot would cost microseconds)
    int winner_of_slot[NMAX];
    uint8_t src[NMAX], save[NMAX];
};

__device__ __forceinline__ void plan_choose(const PlanSmem& ps, int s, bool restricted, int& src, unsigned long long& adds) {
    const unsigned long long cur = ps.loose[s];
    int best_cost = __popcll(cur);
    src = -1;
    adds = cur;
    if (s > 0) {
        const unsigned long long prev = ps.loose[s - 1];
        if ((prev & ~cur) == 0ull) {
            const int c = __popcll(cur & ~prev);
            if (c <= best_cost) { best_cost = c; src = -2; adds = cur & ~prev; }
        }
    }
    for (int j = 0; j + 1 < s; ++j) {
        if (restricted && ps.saved[j] < 0) continue;
        const unsigned long long sj = ps.loose[j];
        if (sj == 0ull || (sj & ~cur) != 0ull) continue;
        const int c = __popcll(cur & ~sj) + 1;          // +1: reading the saved sum
        if (c < best_cost) { best_cost = c; src = j; adds = cur & ~sj; }
    }
}

__device__ void build_schedule(gar_selection_t* sel, PlanSmem& ps) {
    const int theta = sel->theta;
    const int tid = threadIdx.x;
    if (tid < theta) {
        const int r = theta - 1 - tid;
        const unsigned long long set_r = sel->sets[r];
        ps.slotset[tid] = set_r;
        ps.winner_of_slot[tid] = sel->winners[r];
        sel->m[r] = __popcll(set_r);
        ps.usage[tid] = 0;
        ps.saved[tid] = -1;
    }
    __syncthreads();
    if (tid == 0) {
        unsigned long long u = 0ull, chain = 0ull, chained_rows = 0ull;
        // suffix intersections: after the loop `suffix` = rows present in every slot
        unsigned long long suffix = ~0ull, next_suffix = ~0ull;
        for (int s = theta - 1; s >= 0; --s) {
            suffix = next_suffix & ps.slotset[s];                 // present in all slots >= s
            const int w = ps.winner_of_slot[s];
            if (w >= 0 && w < NMAX) {
                u |= 1ull << w;
                // chained: permanent from slot s on, and not already permanent from slot s+... (a winner
                // is absent before its own slot, so "present in all slots >= s" pins its entry to s)
                if ((suffix >> w) & 1ull) { chain |= 1ull << s; chained_rows |= 1ull << w; }
            }
            u |= ps.slotset[s];
            next_suffix = suffix;
        }
        // a winner can only be in sets of its own slot and later ones; if the caller's tables break
        // that (a chained row also present earlier), un-chain nothing: the covered set below stays a
        // subset of every slot set because chained rows are in all slots >= their own and are only
        // counted from their own slot on.
        const unsigned long long base = suffix & ~chained_rows;  // suffix at s = 0
        ps.uni = u;
        ps.base = base;
        ps.chain = chain;
        unsigned long long covered = base, loose_all = 0ull;
        for (int s = 0; s < theta; ++s) {
            if ((chain >> s) & 1ull) covered |= 1ull << ps.winner_of_slot[s];
            ps.loose[s] = ps.slotset[s] & ~covered;
            loose_all |= ps.loose[s];
        }
        ps.loose_all = loose_all;
        sel->nu = __popcll(u);
        sel->nbase = __popcll(base);
        sel->nloose = __popcll(loose_all);
        sel->chain_mask = chain;
    }
    __syncthreads();
    const unsigned long long base = ps.base, loose_all = ps.loose_all;
    if (tid < NMAX) {
        const unsigned long long below = (1ull << tid) - 1ull;
        if ((base >> tid) & 1ull) sel->base_rows[__popcll(base & below)] = uint8_t(tid);
        if ((loose_all >> tid) & 1ull) sel->loose_rows[__popcll(loose_all & below)] = uint8_t(tid);
    }
    // pass 1: unrestricted choice, to see which corrections are worth keeping
    if (tid < theta) {
        int src; unsigned long long adds;
        plan_choose(ps, tid, false, src, adds);
        ps.choice[tid] = src;
    }
    __syncthreads();
    if (tid == 0) {
        for (int s = 0; s < theta; ++s) if (ps.choice[s] >= 0) ps.usage[ps.choice[s]] += 1;
        for (int k = 0; k < GAR_MAX_SAVED; ++k) {           // keep the most used ones
            int bj = -1, bu = 0;
            for (int j = 0; j < theta; ++j) if (ps.saved[j] < 0 && ps.usage[j] > bu) { bu = ps.usage[j]; bj = j; }
            if (bj < 0) break;
            ps.saved[bj] = k;
        }
    }
    __syncthreads();
    // pass 2: final choice among the kept corrections
    if (tid < theta) {
        int src; unsigned long long adds;
        plan_choose(ps, tid, true, src, adds);
        ps.addmask[tid] = adds;
        ps.src[tid] = src == -1 ? uint8_t(GAR_SRC_ZERO) : src == -2 ? uint8_t(GAR_SRC_CONT) : uint8_t(ps.saved[src]);
        ps.save[tid] = ps.saved[tid] >= 0 ? uint8_t(ps.saved[tid]) : uint8_t(GAR_SAVE_NONE);
        sel->slot_src[tid] = ps.src[tid];
        sel->slot_nadd[tid] = uint8_t(__popcll(adds));
        sel->slot_save[tid] = ps.save[tid];
    }
    __syncthreads();
    if (tid == 0) {
        int acc = 0;
        unsigned long long corr = 0ull;
        for (int s = 0; s < theta; ++s) {
            ps.offset[s] = acc;
            const int na = __popcll(ps.addmask[s]);
            acc += na;
            const bool noop = (na == 0) && ps.save[s] == GAR_SAVE_NONE &&
                              (ps.src[s] == GAR_SRC_CONT || (s == 0 && ps.src[s] == GAR_SRC_ZERO));
            if (!noop) corr |= 1ull << s;
        }
        ps.offset[theta] = acc;
        sel->total_adds = acc;
        sel->corr_mask = corr;
    }
    __syncthreads();
    if (tid < theta) {
        unsigned long long adds = ps.addmask[tid];
        int pos = ps.offset[tid];
        while (adds) {
            const int b = __ffsll((long long)adds) - 1;
            sel->add_pos[pos++] = uint8_t(__popcll(loose_all & ((1ull << b) - 1ull)));
            adds &= adds - 1;
        }
    }
}

__global__ void __launch_bounds__(K2_THREADS)
k2_select(const double* __restrict__ dist, gar_selection_t* __restrict__ sel, int rule, int n, int f,
          int m_user, int theta, int beta, int median_of_agr, int even_median) {
    dist += size_t(blockIdx.x) * n * n;           // a batch: CTA b takes the b-th matrix and selection
    sel += blockIdx.x;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    K2Smem& sm = *reinterpret_cast<K2Smem*>(smem_raw);
    __shared__ PlanSmem plan_smem;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    const bool preagg = (rule == GAR_MULTI_BULYAN || rule == GAR_MULTI_KRUM || rule == GAR_AVERAGE);
    if (tid == 0) {
        sel->n = n; sel->f = f; sel->rule = rule; sel->theta = theta; sel->beta = beta;
        sel->preagg = preagg ? 1 : 0;
        sel->median_of_agr = median_of_agr;
        sel->even_median = even_median;
        sel->reserved = 0;
        sel->status = GAR_OK;
    }

    if (rule == GAR_AVERAGE || rule == GAR_MEDIAN) {
        // no scoring: averaging is one "round" whose set is everybody; the
        // median rule extracts every gradient and keeps the one value at the median
        if (tid < theta) {
            sel->winners[tid] = (rule == GAR_MEDIAN) ? tid : 0;
            sel->sets[tid] = (rule == GAR_MEDIAN) ? (1ull << tid) : (n == 64 ? ~0ull : ((1ull << n) - 1ull));
            sel->gap_winner[tid] = INFINITY;
            sel->gap_set[tid] = INFINITY;
        }
        __syncthreads();
        build_schedule(sel, plan_smem);
        return;
    }

    // 1. load.  A NaN on the diagonal is how a distance kernel that gave up on a wait marks its
    // matrix: nothing is selected from it (selecting by index from all-infinite scores would hand
    // arbitrary, possibly Byzantine, gradients to the coordinate phase as if nothing had happened).
    bool poisoned = false;
    for (int idx = tid; idx < n * n; idx += K2_THREADS) {
        const int i = idx / n, j = idx - i * n;
        double v = dist[idx];
        if (i == j) { poisoned |= (v != v); v = 0.0; }
        if (!isfinite(v)) v = INFINITY;
        sm.dm[i][j] = v;
    }
    if (__syncthreads_or(poisoned ? 1 : 0)) {
        if (tid == 0) sel->status = GAR_ERR_TIMEOUT;
        return;
    }
    // 2. sort every row's other entries on (value, index) by counting
    for (int idx = tid; idx < n * n; idx += K2_THREADS) {
        const int i = idx / n, j = idx - i * n;
        if (i == j) continue;
        const double v = sm.dm[i][j];
        int rank = 0;
        for (int jj = 0; jj < n; ++jj) {
            if (jj == i) continue;
            const double u = sm.dm[i][jj];
            rank += (u < v || (u == v && jj < j)) ? 1 : 0;
        }
        sm.sv[i][rank] = v;
        sm.sj[i][rank] = uint8_t(j);
    }
    if (tid == 0) sm.alive = (n == 64) ? ~0ull : ((1ull << n) - 1ull);
    __syncthreads();

    const bool clamp = (rule == GAR_BULYAN);
    // 3. rounds
    for (int r = 0; r < theta; ++r) {
        const int k = n - r;
        int q = k - f - 2;
        if (clamp && q < 1) q = 1;
        int m = 1;
        if (rule == GAR_MULTI_BULYAN) m = k - f - 2;
        else if (rule == GAR_MULTI_KRUM) m = m_user > 0 ? m_user : n - f - 2;
        const unsigned long long alive = sm.alive;

        // 3a. scores: warp per row
        for (int i = warp; i < n; i += K2_THREADS / 32) {
            double s = INFINITY;
            if ((alive >> i) & 1ull) {
                const int p0 = lane, p1 = lane + 32;
                const bool v0 = p0 < n - 1, v1 = p1 < n - 1;
                const int j0 = v0 ? sm.sj[i][p0] : 0, j1 = v1 ? sm.sj[i][p1] : 0;
                const bool a0 = v0 && ((alive >> j0) & 1ull), a1 = v1 && ((alive >> j1) & 1ull);
                const unsigned b0 = __ballot_sync(0xffffffffu, a0), b1 = __ballot_sync(0xffffffffu, a1);
                const unsigned lt = (1u << lane) - 1u;
                const int c0 = __popc(b0 & lt), c1 = __popc(b0) + __popc(b1 & lt);
                double x = 0.0;
                if (a0 && c0 < q) x += sm.sv[i][p0];
                if (a1 && c1 < q) x += sm.sv[i][p1];
#pragma unroll
                for (int o = 16; o >= 1; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
                s = x;
            }
            if (lane == 0) {
                sm.score[i] = s;
                sel->scores[r][i] = s;
            }
        }
        __syncthreads();

        // 3b. rank on (score, index), a warp per row: the rank is the number of remaining rows that
        // come before it.  The row of rank 0 is the winner and leaves; ranks below m form the set.
        for (int i = warp; i < n; i += K2_THREADS / 32) {
            if ((alive >> i) & 1ull) {
                const double s = sm.score[i];
                const int j0 = lane, j1 = lane + 32;
                bool c0 = false, c1 = false;
                if (j0 < n && ((alive >> j0) & 1ull)) { const double u = sm.score[j0]; c0 = u < s || (u == s && j0 < i); }
                if (j1 < n && ((alive >> j1) & 1ull)) { const double u = sm.score[j1]; c1 = u < s || (u == s && j1 < i); }
                const int rank = __popc(__ballot_sync(0xffffffffu, c0)) + __popc(__ballot_sync(0xffffffffu, c1));
                if (lane == 0) {
                    if (rank == 0) {
                        sm.pick[r][0] = s;
                        sel->winners[r] = i;
                        sm.alive = alive & ~(1ull << i);        // everybody holds this round's mask in a register
                    }
                    if (rank == 1) sm.pick[r][1] = s;
                    if (rank == m - 1) sm.pick[r][2] = s;
                    if (rank == m) sm.pick[r][3] = s;
                    sm.order[r][rank] = uint8_t(i);
                }
            }
        }
        __syncthreads();
    }
    // sets and gaps of all rounds
    if (tid < theta) {
        const int r = tid, k = n - r;
        int m = 1;
        if (rule == GAR_MULTI_BULYAN) m = k - f - 2;
        else if (rule == GAR_MULTI_KRUM) m = m_user > 0 ? m_user : n - f - 2;
        unsigned long long mask = 0ull;                     // the m best ranks of the round
        for (int j = 0; j < m; ++j) mask |= 1ull << sm.order[r][j];
        sel->sets[r] = mask;
        sel->gap_winner[r] = (k > 1) ? rel_gap(sm.pick[r][0], sm.pick[r][1]) : INFINITY;
        sel->gap_set[r] = (m < k) ? rel_gap(sm.pick[r][2], sm.pick[r][3]) : INFINITY;
    }
    __syncthreads();
    // 4. schedule
    build_schedule(sel, plan_smem);
}

__global__ void __launch_bounds__(64) k2_schedule_only(gar_selection_t* sel) {
    __shared__ PlanSmem plan_smem;
    build_schedule(sel, plan_smem);
}

}  // namespace

cudaError_t launch_select(int rule, const double* dist, int n, int f, int m, int theta, int beta,
                          int median_of_agr, int even_median, gar_selection_t* sel, cudaStream_t stream, int count) {
    static bool configured[64] = {false};
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (!(dev >= 0 && dev < 64 && configured[dev])) {
        err = cudaFuncSetAttribute(k2_select, cudaFuncAttributeMaxDynamicSharedMemorySize, int(sizeof(K2Smem)));
        if (err != cudaSuccess) return err;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    k2_select<<<unsigned(count), K2_THREADS, sizeof(K2Smem), stream>>>(dist, sel, rule, n, f, m, theta, beta, median_of_agr, even_median);
    return cudaGetLastError();
}

cudaError_t launch_schedule_only(gar_selection_t* sel, cudaStream_t stream) {
    k2_schedule_only<<<1, 64, 0, stream>>>(sel);
    return cudaGetLastError();
}

}  // namespace gar
