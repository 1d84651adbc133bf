// Coordinate phase (Algorithm 1, multi-Bulyan: M = Median(G^ext); per coordinate
// the beta entries of G^agr closest to M; their average), one streaming pass.
//
// G^ext and G^agr are never written to memory.  For every coordinate a thread
// loads the gradients it needs straight from the n x d block and rebuilds
//    e[s] = G[winner of round theta-1-s]           (G^ext, reversed round order)
//    a[s] = mean of G over that round's set        (G^agr)
// in registers.  Rounds are visited last-to-first ("slots") because the sets
// shrink by one gradient per round: the running sum T then only grows,
// T_s = T_{s-1} + (rows the earlier round has on top), and no value is ever
// subtracted.  In the usual case (sets[r] = sets[r+1] + {winner_r}, "nested")
// the row added at slot s is exactly the winner whose value is e[s], so every
// needed row is loaded exactly once: |sets[0]| loads per coordinate.  Any other
// set structure runs the general schedule (restart flags + row lists).
// The median is a Batcher odd-even merge sorting network over registers, pruned
// by the compiler to the comparators the middle output depends on; the beta
// closest values are found by beta passes of arg-min over |a - M|.
//
// P is the compiled slot count (>= theta): slots >= theta are padding that is
// never loaded; the median padding is split between -inf and +inf so that the
// lower median of the theta real values sits at index (P-1)/2.
#pragma once
#include <math_constants.h>

#include <utility>

#include "gar_internal.cuh"

namespace gar {

constexpr int K3_THREADS = 256;

struct K3Plan {
    int     theta, beta, median_of_agr, nested, base_count, lo_pads;
    int64_t woff[GAR_MAX_N];       // slot -> winner row offset (elements)
    float   inv_m[GAR_MAX_N];      // slot -> 1/|set|
    int64_t base_off[GAR_MAX_N];   // slot 0 rows
    int     seg_start[GAR_MAX_N + 1];
    uint8_t restart[GAR_MAX_N];
    uint8_t prog_rows[GAR_MAX_N * GAR_MAX_N];
};

template <int V> struct VecT;
template <> struct VecT<1> { using type = float; };
template <> struct VecT<2> { using type = float2; };
template <> struct VecT<4> { using type = float4; };

template <int V> __device__ __forceinline__ void load_vec(const float* p, float (&x)[V]) {
    if constexpr (V == 1) { x[0] = __ldg(p); }
    else if constexpr (V == 2) { float2 t = __ldg(reinterpret_cast<const float2*>(p)); x[0] = t.x; x[1] = t.y; }
    else { float4 t = __ldg(reinterpret_cast<const float4*>(p)); x[0] = t.x; x[1] = t.y; x[2] = t.z; x[3] = t.w; }
}
template <int V> __device__ __forceinline__ void store_vec(float* p, const float (&x)[V]) {
    if constexpr (V == 1) { *p = x[0]; }
    else if constexpr (V == 2) { *reinterpret_cast<float2*>(p) = make_float2(x[0], x[1]); }
    else { *reinterpret_cast<float4*>(p) = make_float4(x[0], x[1], x[2], x[3]); }
}

__device__ __forceinline__ void cmpswap(float& lo, float& hi) {
    const float a = lo, b = hi;
    lo = fminf(a, b);
    hi = fmaxf(a, b);
}

// Comparator list of Batcher's odd-even merge sort for any N (ascending), built
// at compile time and pruned to the comparators that the output at index
// (N-1)/2 depends on (walked backwards from that output).
template <int N> struct MedianNet {
    static constexpr int MAXC = (N < 4) ? 8 : N * 10;
    struct Data {
        int a[MAXC];
        int b[MAXC];
        int count;
    };
    static constexpr Data build() {
        Data all{};
        int cnt = 0;
        for (int p = 1; p < N; p *= 2)
            for (int k = p; k >= 1; k /= 2)
                for (int j = k % p; j + k < N; j += 2 * k)
                    for (int i = 0; i < k; ++i)
                        if (i + j + k < N && (i + j) / (2 * p) == (i + j + k) / (2 * p)) {
                            all.a[cnt] = i + j;
                            all.b[cnt] = i + j + k;
                            ++cnt;
                        }
        bool live[N > 0 ? N : 1] = {};
        live[(N - 1) / 2] = true;
        bool keep[MAXC] = {};
        for (int c = cnt - 1; c >= 0; --c) {
            if (live[all.a[c]] || live[all.b[c]]) {
                keep[c] = true;
                live[all.a[c]] = true;
                live[all.b[c]] = true;
            }
        }
        Data out{};
        int oc = 0;
        for (int c = 0; c < cnt; ++c)
            if (keep[c]) { out.a[oc] = all.a[c]; out.b[oc] = all.b[c]; ++oc; }
        out.count = oc;
        return out;
    }
    static constexpr Data data = build();
};

template <int V> __device__ __forceinline__ void cmpswap_vec(float (&lo)[V], float (&hi)[V]) {
#pragma unroll
    for (int v = 0; v < V; ++v) cmpswap(lo[v], hi[v]);
}

template <int N, int V, size_t... C>
__device__ __forceinline__ void median_network_apply(float (&x)[N][V], std::index_sequence<C...>) {
    (cmpswap_vec<V>(x[MedianNet<N>::data.a[C]], x[MedianNet<N>::data.b[C]]), ...);
}

// After the call x[(N-1)/2] holds the lower median; other entries are unspecified.
template <int N, int V> __device__ __forceinline__ void median_network(float (&x)[N][V]) {
    median_network_apply<N, V>(x, std::make_index_sequence<MedianNet<N>::data.count>{});
}

__device__ __forceinline__ void load_plan(K3Plan& plan, const gar_selection_t* __restrict__ sel, int64_t ld, int P) {
    const int tid = threadIdx.x;
    const int theta = sel->theta;
    if (tid == 0) {
        plan.theta = theta;
        plan.beta = sel->beta;
        plan.median_of_agr = sel->median_of_agr;
        plan.nested = sel->nested;
        plan.base_count = sel->base_count;
        plan.lo_pads = (P - 1) / 2 - (theta - 1) / 2;
    }
    for (int s = tid; s < theta; s += blockDim.x) {
        const int r = theta - 1 - s;
        plan.woff[s] = int64_t(sel->winners[r]) * ld;
        plan.inv_m[s] = 1.0f / float(sel->m[r]);
        plan.restart[s] = sel->restart[s];
    }
    for (int s = tid; s <= theta; s += blockDim.x) plan.seg_start[s] = sel->seg_start[s];
    for (int b = tid; b < sel->base_count; b += blockDim.x) plan.base_off[b] = int64_t(sel->base_rows[b]) * ld;
    if (sel->preagg && !sel->nested) {
        const int total = sel->seg_start[theta];
        for (int k = tid; k < total; k += blockDim.x) plan.prog_rows[k] = sel->prog_rows[k];
    }
}

// Coordinates [t_begin, t_end), V per thread; (t_end - t_begin) % V == 0 and the
// V-vectors at g + row*ld + t and out + t are naturally aligned.
template <int P, bool PREAGG, int V>
__global__ void __launch_bounds__(K3_THREADS)
k3_coordinate(const float* __restrict__ g, int64_t t_begin, int64_t t_end, int64_t ld,
              const gar_selection_t* __restrict__ sel, float* __restrict__ out) {
    __shared__ K3Plan plan;
    load_plan(plan, sel, ld, P);
    __syncthreads();
    const int theta = plan.theta;
    const int beta = plan.beta;
    const float inv_beta = 1.0f / float(beta);
    const int lo_pads = plan.lo_pads;
    const bool med_agr = plan.median_of_agr != 0;

    const int64_t nvec = (t_end - t_begin) / V;
    for (int64_t vi = int64_t(blockIdx.x) * K3_THREADS + threadIdx.x; vi < nvec;
         vi += int64_t(gridDim.x) * K3_THREADS) {
        const int64_t t = t_begin + vi * V;
        const float* gt = g + t;
        float e[P][V], a[P][V];
#pragma unroll
        for (int s = 0; s < P; ++s) {
#pragma unroll
            for (int v = 0; v < V; ++v) { e[s][v] = 0.0f; a[s][v] = 0.0f; }
        }

        if constexpr (PREAGG) {
            float T[V];
            if (plan.nested) {
                float x[V];
                load_vec<V>(gt + plan.base_off[0], x);
#pragma unroll
                for (int v = 0; v < V; ++v) { e[0][v] = x[v]; T[v] = x[v]; }
                const int bc = plan.base_count;
#pragma unroll 4
                for (int b = 1; b < bc; ++b) {
                    load_vec<V>(gt + plan.base_off[b], x);
#pragma unroll
                    for (int v = 0; v < V; ++v) T[v] += x[v];
                }
                const float im0 = plan.inv_m[0];
#pragma unroll
                for (int v = 0; v < V; ++v) a[0][v] = T[v] * im0;
#pragma unroll
                for (int s = 1; s < P; ++s) {
                    if (s < theta) {
                        load_vec<V>(gt + plan.woff[s], x);
                        const float im = plan.inv_m[s];
#pragma unroll
                        for (int v = 0; v < V; ++v) { T[v] += x[v]; e[s][v] = x[v]; a[s][v] = T[v] * im; }
                    }
                }
            } else {
#pragma unroll
                for (int v = 0; v < V; ++v) T[v] = 0.0f;
#pragma unroll
                for (int s = 0; s < P; ++s) {
                    if (s < theta) {
                        float x[V];
                        if (plan.restart[s]) {
#pragma unroll
                            for (int v = 0; v < V; ++v) T[v] = 0.0f;
                        }
                        const int k1 = plan.seg_start[s + 1];
                        for (int k = plan.seg_start[s]; k < k1; ++k) {
                            load_vec<V>(gt + int64_t(plan.prog_rows[k]) * ld, x);
#pragma unroll
                            for (int v = 0; v < V; ++v) T[v] += x[v];
                        }
                        load_vec<V>(gt + plan.woff[s], x);
                        const float im = plan.inv_m[s];
#pragma unroll
                        for (int v = 0; v < V; ++v) { e[s][v] = x[v]; a[s][v] = T[v] * im; }
                    }
                }
            }
        } else {
#pragma unroll
            for (int s = 0; s < P; ++s) {
                if (s < theta) {
                    float x[V];
                    load_vec<V>(gt + plan.woff[s], x);
#pragma unroll
                    for (int v = 0; v < V; ++v) { e[s][v] = x[v]; a[s][v] = x[v]; }
                }
            }
        }

        // median of the theta real values (lower middle), padding split around them
        float srt[P][V];
#pragma unroll
        for (int s = 0; s < P; ++s) {
#pragma unroll
            for (int v = 0; v < V; ++v) {
                const float real = (PREAGG && med_agr) ? a[s][v] : e[s][v];
                const float pad = (s - theta < lo_pads) ? -CUDART_INF_F : CUDART_INF_F;
                srt[s][v] = (s < theta) ? real : pad;
            }
        }
        median_network<P, V>(srt);
        float key[P][V];
#pragma unroll
        for (int s = 0; s < P; ++s) {
#pragma unroll
            for (int v = 0; v < V; ++v)
                key[s][v] = (s < theta) ? fabsf(a[s][v] - srt[(P - 1) / 2][v]) : CUDART_INF_F;
        }

        // beta passes of arg-min; equal keys go to the earliest round = highest slot
        float sum[V];
#pragma unroll
        for (int v = 0; v < V; ++v) sum[v] = 0.0f;
        for (int b = 0; b < beta; ++b) {
#pragma unroll
            for (int v = 0; v < V; ++v) {
                float best = CUDART_INF_F, ba = 0.0f;
                int bi = -1;
#pragma unroll
                for (int s = P - 1; s >= 0; --s) {
                    const bool take = (s < theta) && (key[s][v] < best || bi < 0);
                    best = take ? key[s][v] : best;
                    ba = take ? a[s][v] : ba;
                    bi = take ? s : bi;
                }
                sum[v] += ba;
                if (b + 1 < beta) {
#pragma unroll
                    for (int s = 0; s < P; ++s) key[s][v] = (s == bi) ? CUDART_INF_F : key[s][v];
                }
            }
        }
        float res[V];
#pragma unroll
        for (int v = 0; v < V; ++v) res[v] = sum[v] * inv_beta;
        store_vec<V>(out + t, res);
    }
}

template <int P>
cudaError_t launch_k3_p(const float* g, int64_t d, int64_t ld, const gar_selection_t* sel, int preagg,
                        int vec, float* out, int sm_count, cudaStream_t stream);

}  // namespace gar
