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
    double   pick[4];             // s(1), s(2), s(m), s(m+1)
    unsigned set_bits[2];
    unsigned long long alive;
    int      winner;
};

__device__ __forceinline__ double rel_gap(double lo, double hi) {
    if (!isfinite(hi)) return isfinite(lo) ? INFINITY : 0.0;
    if (hi <= 0.0) return 0.0;
    return (hi - lo) / hi;
}

// Derive the coordinate kernel's schedule from winners[] and sets[] (see gar.h).
// Slots are rounds in reverse: slot s = theta-1-r, so that the running sum only
// ever grows: slot 0 sums the last round's set, slot s adds what round
// theta-1-s has on top of the following round.
__device__ void build_schedule(gar_selection_t* sel, int* counts /* shared, NMAX+1 */) {
    const int theta = sel->theta;
    const int tid = threadIdx.x;
    if (tid < theta) {
        const int s = tid, r = theta - 1 - s;
        const uint64_t cur = sel->sets[r];
        sel->m[r] = __popcll(cur);
        uint64_t adds = cur;
        int restart = 1;
        if (s > 0) {
            const uint64_t prev = sel->sets[r + 1];
            if ((prev & ~cur) == 0ull) { adds = cur & ~prev; restart = 0; }
        }
        sel->restart[s] = uint8_t(restart);
        counts[s] = __popcll(adds);
    }
    __syncthreads();
    if (tid == 0) {
        int acc = 0;
        for (int s = 0; s < theta; ++s) { sel->seg_start[s] = acc; acc += counts[s]; }
        sel->seg_start[theta] = acc;
    }
    __syncthreads();
    if (tid < theta) {
        const int s = tid, r = theta - 1 - s;
        const uint64_t cur = sel->sets[r];
        uint64_t adds = cur;
        if (s > 0 && !sel->restart[s]) adds = cur & ~sel->sets[r + 1];
        int pos = sel->seg_start[s];
        const int w = sel->winners[r];
        // the winner first (slot 0 relies on it), then ascending
        if (w >= 0 && w < NMAX && ((adds >> w) & 1ull)) { sel->prog_rows[pos++] = uint8_t(w); adds &= ~(1ull << w); }
        while (adds) { int b = __ffsll((long long)adds) - 1; sel->prog_rows[pos++] = uint8_t(b); adds &= adds - 1; }
    }
    __syncthreads();
    if (tid == 0) {
        int nested = sel->preagg ? 1 : 0;
        const int wl = sel->winners[theta - 1];
        const int bc = sel->seg_start[1] - sel->seg_start[0];
        if (!(wl >= 0 && wl < NMAX && ((sel->sets[theta - 1] >> wl) & 1ull))) nested = 0;
        for (int s = 1; s < theta && nested; ++s) {
            const int r = theta - 1 - s;
            if (sel->restart[s] || sel->seg_start[s + 1] - sel->seg_start[s] != 1 ||
                sel->prog_rows[sel->seg_start[s]] != sel->winners[r])
                nested = 0;
        }
        sel->nested = nested;
        sel->base_count = bc;
        for (int b = 0; b < bc && b < NMAX; ++b) sel->base_rows[b] = sel->prog_rows[b];
    }
}

__global__ void __launch_bounds__(K2_THREADS)
k2_select(const double* __restrict__ dist, gar_selection_t* __restrict__ sel, int rule, int n, int f,
          int m_user, int theta, int beta, int median_of_agr) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    K2Smem& sm = *reinterpret_cast<K2Smem*>(smem_raw);
    __shared__ int counts[NMAX + 1];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    const bool preagg = (rule == GAR_MULTI_BULYAN || rule == GAR_MULTI_KRUM || rule == GAR_AVERAGE);
    if (tid == 0) {
        sel->n = n; sel->f = f; sel->rule = rule; sel->theta = theta; sel->beta = beta;
        sel->preagg = preagg ? 1 : 0;
        sel->median_of_agr = median_of_agr;
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
        build_schedule(sel, counts);
        return;
    }

    // 1. load
    for (int idx = tid; idx < n * n; idx += K2_THREADS) {
        const int i = idx / n, j = idx - i * n;
        double v = dist[idx];
        if (!isfinite(v)) v = INFINITY;
        if (i == j) v = 0.0;
        sm.dm[i][j] = v;
    }
    __syncthreads();
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

        // 3b. rank on (score, index); winner, set, gaps
        if (tid < 64) {
            bool in_set = false;
            if (tid < n && ((alive >> tid) & 1ull)) {
                const double s = sm.score[tid];
                int rank = 0;
                for (int j = 0; j < n; ++j) {
                    if (!((alive >> j) & 1ull)) continue;
                    const double u = sm.score[j];
                    rank += (u < s || (u == s && j < tid)) ? 1 : 0;
                }
                if (rank == 0) { sm.winner = tid; sm.pick[0] = s; }
                if (rank == 1) sm.pick[1] = s;
                if (rank == m - 1) sm.pick[2] = s;
                if (rank == m) sm.pick[3] = s;
                in_set = rank < m;
            }
            const unsigned bits = __ballot_sync(0xffffffffu, in_set);
            if (lane == 0) sm.set_bits[warp] = bits;
        }
        __syncthreads();
        if (tid == 0) {
            const int w = sm.winner;
            sel->winners[r] = w;
            sel->sets[r] = (uint64_t(sm.set_bits[1]) << 32) | uint64_t(sm.set_bits[0]);
            sel->gap_winner[r] = (k > 1) ? rel_gap(sm.pick[0], sm.pick[1]) : INFINITY;
            sel->gap_set[r] = (m < k) ? rel_gap(sm.pick[2], sm.pick[3]) : INFINITY;
            sm.alive = alive & ~(1ull << w);
        }
        __syncthreads();
    }
    // 4. schedule
    build_schedule(sel, counts);
}

__global__ void __launch_bounds__(64) k2_schedule_only(gar_selection_t* sel) {
    __shared__ int counts[NMAX + 1];
    build_schedule(sel, counts);
}

}  // namespace

cudaError_t launch_select(int rule, const double* dist, int n, int f, int m, int theta, int beta,
                          int median_of_agr, gar_selection_t* sel, cudaStream_t stream) {
    static bool configured[64] = {false};
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (!(dev >= 0 && dev < 64 && configured[dev])) {
        err = cudaFuncSetAttribute(k2_select, cudaFuncAttributeMaxDynamicSharedMemorySize, int(sizeof(K2Smem)));
        if (err != cudaSuccess) return err;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    k2_select<<<1, K2_THREADS, sizeof(K2Smem), stream>>>(dist, sel, rule, n, f, m, theta, beta, median_of_agr);
    return cudaGetLastError();
}

cudaError_t launch_schedule_only(gar_selection_t* sel, cudaStream_t stream) {
    k2_schedule_only<<<1, 64, 0, stream>>>(sel);
    return cudaGetLastError();
}

}  // namespace gar
