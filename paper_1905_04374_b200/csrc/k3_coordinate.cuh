// Coordinate phase (Algorithm 1, multi-Bulyan: M = Median(G^ext); per coordinate
// the beta entries of G^agr closest to M; their average), one streaming pass.
//
// G^ext and G^agr are never written to memory.  For every coordinate a thread
// loads the gradients it needs straight from the n x d block and rebuilds
//    e[s] = G[winner of round theta-1-s]           (G^ext, reversed round order)
//    a[s] = mean of G over that round's set        (G^agr)
// in registers ("slot" s = round theta-1-s).
//  * Rules without pre-aggregation (Bulyan, Median, Krum: a = e) load the theta
//    winner rows, one load each.
//  * Pre-aggregating rules (multi-Bulyan, multi-Krum, averaging) follow the
//    summation plan of the selection kernel (layout in gar.h):
//       T_s = sum(base rows) + sum(chained winners up to slot s) + C_s.
//    Base rows are added as they arrive; a chained winner's value is e[s], already
//    in a register, so the chain costs one add per slot; only the few "loose"
//    gradients are parked in a shared-memory column private to the thread
//    (dynamic indexing without local memory, no barrier) and summed into C_s by
//    the plan.  Every needed gradient is loaded exactly once, except a winner
//    that is also loose (twice, the second time from L1).
// The median is a Batcher odd-even merge network over registers, pruned at
// compile time to the comparators the middle output depends on; the beta
// closest values are found from the beta-th smallest |a - M| (min/max only)
// and 0/1 masks, with arg-min passes as the general fallback.
//
// P is the compiled slot count.  EXACT kernels have theta == P at compile time;
// the others take theta <= P at run time: slots >= theta are padding that is
// never loaded, and the median padding is split between -inf and +inf so that
// the lower median of the theta real values sits at index (P-1)/2.
#pragma once
#include <math_constants.h>

#include <utility>

#include "gar_internal.cuh"

namespace gar {

constexpr int K3_THREADS = 256;
constexpr int K3_LOOSE_CAP = 32;      // loose gradients parked in shared memory; more: read from global

struct K3Plan {
    int      theta, beta, median_of_agr, lo_pads, nbase, nloose, loose_in_smem, even_mean, median_only;
    unsigned long long chain_mask, corr_mask;
    int64_t  woff[GAR_MAX_N];       // slot -> winner row offset (elements)
    int64_t  boff[GAR_MAX_N];       // base row offsets
    int64_t  loff[GAR_MAX_N];       // loose row offsets
    float    inv_m[GAR_MAX_N];      // slot -> 1/|set|
    uint8_t  src[GAR_MAX_N], save[GAR_MAX_N], nadd[GAR_MAX_N];
    uint8_t  add_pos[GAR_MAX_N * GAR_MAX_N];
};

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
template <int V> __device__ __forceinline__ void read_vec(const float* p, float (&x)[V]) {
    if constexpr (V == 1) { x[0] = *p; }
    else if constexpr (V == 2) { float2 t = *reinterpret_cast<const float2*>(p); x[0] = t.x; x[1] = t.y; }
    else { float4 t = *reinterpret_cast<const float4*>(p); x[0] = t.x; x[1] = t.y; x[2] = t.z; x[3] = t.w; }
}

// A coordinate's result goes out: the aggregate, and/or the fused SGD step (v <- mu v + g, x <- x - lr v).
template <int V> __device__ __forceinline__ void k3_store(const K3Out& o, int64_t t, const float (&res)[V]) {
    if (o.out) store_vec<V>(o.out + t, res);
    if (o.x) {
        float x[V], step[V];
        read_vec<V>(o.x + t, x);
        if (o.v) {
            float v[V];
            read_vec<V>(o.v + t, v);
#pragma unroll
            for (int k = 0; k < V; ++k) { v[k] = fmaf(o.mu, v[k], res[k]); step[k] = v[k]; }
            store_vec<V>(o.v + t, v);
        } else {
#pragma unroll
            for (int k = 0; k < V; ++k) step[k] = res[k];
        }
#pragma unroll
        for (int k = 0; k < V; ++k) x[k] = fmaf(-o.lr, step[k], x[k]);
        store_vec<V>(o.x + t, x);
    }
}
// Nothing usable was computed: the aggregate says so; the model and its momentum stay as they are.
__device__ __forceinline__ void k3_store_nan(const K3Out& o, int64_t t) {
    if (o.out) o.out[t] = CUDART_NAN_F;
}

// V consecutive gradient elements starting at element `idx` (naturally aligned for V elements),
// widened to fp32: fp32 elements by default, 16-bit ones for dtype GAR_BF16 / GAR_F16.
template <int V> __device__ __forceinline__ void load_grad(const float* g, int64_t idx, int dtype, float (&x)[V]) {
    if (dtype == GAR_F32) { load_vec<V>(g + idx, x); return; }
    const unsigned short* h = reinterpret_cast<const unsigned short*>(g) + idx;
    if constexpr (V == 1) {
        x[0] = widen16(__ldg(h), dtype);
    } else if constexpr (V == 2) {
        const unsigned u = __ldg(reinterpret_cast<const unsigned*>(h));
        x[0] = widen16(static_cast<unsigned short>(u & 0xffffu), dtype);
        x[1] = widen16(static_cast<unsigned short>(u >> 16), dtype);
    } else {
        const uint2 u = __ldg(reinterpret_cast<const uint2*>(h));
        x[0] = widen16(static_cast<unsigned short>(u.x & 0xffffu), dtype);
        x[1] = widen16(static_cast<unsigned short>(u.x >> 16), dtype);
        x[2] = widen16(static_cast<unsigned short>(u.y & 0xffffu), dtype);
        x[3] = widen16(static_cast<unsigned short>(u.y >> 16), dtype);
    }
}

__device__ __forceinline__ void prefetch_l1(const void* p) {
    asm volatile("prefetch.global.L1 [%0];" ::"l"(p));
}

__device__ __forceinline__ void cmpswap(float& lo, float& hi) {
    const float a = lo, b = hi;
    lo = fminf(a, b);
    hi = fmaxf(a, b);
}

// Comparator list of Batcher's odd-even merge sort for any N (ascending), built
// at compile time and pruned to the comparators that the output at index
// (N-1)/2 -- and, for even N, the one at N/2 -- depends on (walked backwards from
// those outputs): the lower and the upper middle value.
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
        live[N / 2] = true;
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

// After the call x[(N-1)/2] holds the lower and x[N/2] the upper middle value; other entries are unspecified.
template <int N, int V> __device__ __forceinline__ void median_network(float (&x)[N][V]) {
    median_network_apply<N, V>(x, std::make_index_sequence<MedianNet<N>::data.count>{});
}

// Last part of a coordinate's work, on V coordinates at once: M = median of the theta real values
// of e (of a when median_of_a; for an even count the lower middle value, or the mean of the two
// middle ones when even_mean), then the average of the beta values of a closest to M
// (Algorithm 1, multi-Bulyan: Median, Argpartition, Average) -- or M itself when median_only (the
// Median rule).  e and a hold P slots of which the first theta are real; e is destroyed.
template <int P, int V>
__device__ __forceinline__ void k3_finish(float (&e)[P][V], float (&a)[P][V], int theta, int beta, float inv_beta,
                                          int lo_pads, bool median_of_a, bool even_mean, bool median_only,
                                          float (&res)[V]) {
    // median of the theta real values (lower middle), padding split around them
    float srt[P][V];
#pragma unroll
    for (int s = 0; s < P; ++s) {
#pragma unroll
        for (int v = 0; v < V; ++v) {
            const float real = median_of_a ? a[s][v] : e[s][v];
            const float pad = (s - theta < lo_pads) ? -CUDART_INF_F : CUDART_INF_F;
            srt[s][v] = (s < theta) ? real : pad;
        }
    }
    median_network<P, V>(srt);
    // the real values sit at sorted positions lo_pads .. lo_pads + theta - 1: the lower middle one
    // at (P-1)/2 and, for an even theta (then P is even too), the upper one at P/2
    float med[V];
    const bool two = even_mean && (theta & 1) == 0;
#pragma unroll
    for (int v = 0; v < V; ++v)
        med[v] = two ? 0.5f * srt[(P - 1) / 2][v] + 0.5f * srt[P / 2][v] : srt[(P - 1) / 2][v];
    if (median_only) {
#pragma unroll
        for (int v = 0; v < V; ++v) res[v] = med[v];
        return;
    }
    float key[P][V];
#pragma unroll
    for (int s = 0; s < P; ++s) {
#pragma unroll
        for (int v = 0; v < V; ++v)
            key[s][v] = (s < theta) ? fabsf(a[s][v] - med[v]) : CUDART_INF_F;
    }

    // The beta smallest keys.  beta == 1: the minimum key, then one scan that keeps the
    // value of the highest slot holding it.  beta == 2, 3: the beta-th smallest key tau is
    // found with min/max only and the values with key <= tau are summed with a 0/1 mask; if
    // more values tie at tau than there is room for, or for larger beta, beta passes of
    // arg-min pick them one by one.  Equal keys go to the earliest round = highest slot.
    float sum[V];
    bool need_passes = beta > 3;
    if (beta == 1) {
#pragma unroll
        for (int v = 0; v < V; ++v) {
            float best = key[0][v];
#pragma unroll
            for (int s = 1; s < P; ++s) best = fminf(best, key[s][v]);
            float ba = a[0][v];
#pragma unroll
            for (int s = 1; s < P; ++s) ba = (key[s][v] == best) ? a[s][v] : ba;
            sum[v] = ba;
        }
    } else if (!need_passes) {
#pragma unroll
        for (int v = 0; v < V; ++v) {
            float t1 = CUDART_INF_F, t2 = CUDART_INF_F, t3 = CUDART_INF_F;   // three smallest keys so far
#pragma unroll
            for (int s = 0; s < P; ++s) {
                const float k = key[s][v];
                const float x = fmaxf(t1, k);
                t1 = fminf(t1, k);
                const float y = fmaxf(t2, x);
                t2 = fminf(t2, x);
                t3 = fminf(t3, y);
            }
            const float tau = beta == 2 ? t2 : t3;
            float s_le = 0.0f, c_le = 0.0f;
#pragma unroll
            for (int s = 0; s < P; ++s) {
                const float le = key[s][v] <= tau ? 1.0f : 0.0f;
                s_le = fmaf(le, a[s][v], s_le);
                c_le += le;
            }
            sum[v] = s_le;
            // c_le > beta: several keys tie at tau and not all of them fit
            // (a non-finite tau or value also lands here)
            if (!(c_le == float(beta)) || !(fabsf(s_le) <= 3.0e38f)) need_passes = true;
        }
    }
    if (need_passes) {
#pragma unroll
        for (int v = 0; v < V; ++v) sum[v] = 0.0f;
        for (int b = 0; b < beta; ++b) {
#pragma unroll
            for (int v = 0; v < V; ++v) {
                float best = key[P - 1][v], ba = a[P - 1][v];
                int bi = P - 1;
#pragma unroll
                for (int s = P - 2; s >= 0; --s) {
                    const bool take = key[s][v] < best;
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
    }
#pragma unroll
    for (int v = 0; v < V; ++v) res[v] = sum[v] * inv_beta;
}

// Checked by every CTA of a coordinate kernel before it forms an address from the selection: the
// status the selection kernel left, and that the tables agree with the arguments the host chose
// the kernel by (theta, pre-aggregation) and only name gradients below n.  The whole CTA calls it;
// the answer (a gar_status_t) is the same in every thread.
__device__ __forceinline__ int k3_check(const gar_selection_t* __restrict__ sel, int n, int theta, bool preagg) {
    const int tid = threadIdx.x, nthreads = blockDim.x;
    const int status = sel->status;
    bool bad = n < 1 || n > GAR_MAX_N || theta < 1 || theta > GAR_MAX_N;
    bad |= sel->theta != theta || (sel->preagg != 0) != preagg || sel->beta < 1 || sel->beta > theta;
    const int nbase = sel->nbase, nloose = sel->nloose, nadds = sel->total_adds;
    if (preagg) bad |= nbase < 0 || nbase > n || nloose < 0 || nloose > n || nadds < 0 || nadds > GAR_MAX_N * GAR_MAX_N;
    if (!bad && status == GAR_OK) {
        for (int s = tid; s < theta; s += nthreads) {
            bad |= unsigned(sel->winners[s]) >= unsigned(n);
            if (preagg) {
                bad |= sel->m[s] < 1 || sel->m[s] > n;
                const int src = sel->slot_src[s], sv = sel->slot_save[s];
                bad |= !(src == GAR_SRC_ZERO || src == GAR_SRC_CONT || src < GAR_MAX_SAVED);
                bad |= !(sv == GAR_SAVE_NONE || sv < GAR_MAX_SAVED);
            }
        }
        if (preagg) {
            for (int k = tid; k < nbase; k += nthreads) bad |= sel->base_rows[k] >= n;
            for (int k = tid; k < nloose; k += nthreads) bad |= sel->loose_rows[k] >= n;
            for (int k = tid; k < nadds; k += nthreads) bad |= sel->add_pos[k] >= nloose;
            if (tid == 0) {
                int total = 0;
                for (int s = 0; s < theta; ++s) total += sel->slot_nadd[s];
                bad |= total != nadds;
            }
        }
    }
    const int any_bad = __syncthreads_or(bad ? 1 : 0);
    if (status != GAR_OK) return status;
    return any_bad ? GAR_ERR_INVALID_ARG : GAR_OK;
}

__device__ __forceinline__ void load_plan(K3Plan& plan, const gar_selection_t* __restrict__ sel, int64_t ld, int P,
                                          bool preagg, int loose_cap) {
    const int tid = threadIdx.x;
    const int theta = sel->theta;
    if (tid == 0) {
        plan.theta = theta;
        plan.beta = sel->beta;
        plan.median_of_agr = sel->median_of_agr;
        plan.lo_pads = (P - 1) / 2 - (theta - 1) / 2;
        plan.nbase = sel->nbase;
        plan.nloose = sel->nloose;
        plan.loose_in_smem = sel->nloose <= loose_cap ? 1 : 0;
        plan.even_mean = sel->even_median == GAR_EVEN_MEDIAN_MEAN ? 1 : 0;
        plan.median_only = sel->rule == GAR_MEDIAN ? 1 : 0;
        plan.chain_mask = sel->chain_mask;
        plan.corr_mask = sel->corr_mask;
    }
    for (int s = tid; s < theta; s += blockDim.x) {
        const int r = theta - 1 - s;
        plan.woff[s] = int64_t(sel->winners[r]) * ld;
        plan.inv_m[s] = 1.0f / float(sel->m[r]);
        plan.src[s] = sel->slot_src[s];
        plan.save[s] = sel->slot_save[s];
        plan.nadd[s] = sel->slot_nadd[s];
    }
    if (preagg) {
        for (int u = tid; u < sel->nbase; u += blockDim.x) plan.boff[u] = int64_t(sel->base_rows[u]) * ld;
        for (int u = tid; u < sel->nloose; u += blockDim.x) plan.loff[u] = int64_t(sel->loose_rows[u]) * ld;
        for (int k = tid; k < sel->total_adds; k += blockDim.x) plan.add_pos[k] = sel->add_pos[k];
    }
}

// Coordinates [t_begin, t_end), V per thread; (t_end - t_begin) % V == 0 and the
// V-vectors at g + row*ld + t and out + t are naturally aligned.
// Dynamic shared memory (PREAGG only): (loose_cap + GAR_MAX_SAVED) * blockDim * V floats.
// bx, gx: this CTA's place among the CTAs that work on the problem.
template <int P, bool EXACT, bool PREAGG, int V>
__device__ __forceinline__ void k3_coordinate_body(const float* __restrict__ g, const int n, const int theta_arg, const int64_t t_begin,
                                                   const int64_t t_end, const int64_t ld, gar_selection_t* __restrict__ sel,
                                                   const K3Out& out, const int loose_cap, const int dtype, const unsigned bx,
                                                   const unsigned gx) {
    __shared__ K3Plan plan;
    extern __shared__ __align__(16) float k3_dyn[];
    const int status = k3_check(sel, n, theta_arg, PREAGG);
    if (status != GAR_OK) {                       // nothing usable: the output says so
        for (int64_t t = t_begin + int64_t(bx) * blockDim.x + threadIdx.x; t < t_end; t += int64_t(gx) * blockDim.x)
            k3_store_nan(out, t);
        if (bx == 0 && threadIdx.x == 0 && sel->status == GAR_OK) sel->status = status;
        return;
    }
    load_plan(plan, sel, ld, P, PREAGG, loose_cap);
    __syncthreads();
    const int theta = EXACT ? P : plan.theta;
    const int beta = plan.beta;
    const float inv_beta = 1.0f / float(beta);
    const int lo_pads = EXACT ? 0 : plan.lo_pads;
    const bool med_agr = plan.median_of_agr != 0;
    const bool even_mean = plan.even_mean != 0, median_only = plan.median_only != 0;
    const int nthreads = blockDim.x;
    // this thread's private columns: loose value u at xcol[u*stride], saved sum k at tcol[k*stride]
    const int stride = nthreads * V;
    float* const xcol = k3_dyn + threadIdx.x * V;
    float* const tcol = xcol + size_t(loose_cap) * stride;
    const unsigned long long chain_mask = plan.chain_mask, corr_mask = plan.corr_mask;

    const int64_t nvec = (t_end - t_begin) / V;
    for (int64_t vi = int64_t(bx) * nthreads + threadIdx.x; vi < nvec;
         vi += int64_t(gx) * nthreads) {
        const int64_t t = t_begin + vi * V;
        const int esh = dtype == GAR_F32 ? 2 : 1;             // log2 of the element size
        float e[P][V], a[P][V];
#pragma unroll
        for (int s = 0; s < P; ++s) {
            if (s < theta) {
                load_grad<V>(g, t + plan.woff[s], dtype, e[s]);
            } else {
#pragma unroll
                for (int v = 0; v < V; ++v) e[s][v] = 0.0f;
            }
        }
        // few slots: the kernel waits on memory more than it computes, so pull the next
        // iteration's lines into L1 meanwhile (with many slots the extra instructions cost more)
        const int64_t vnext = vi + int64_t(gx) * nthreads;
        if (P <= 12 && vnext < nvec) {
            const char* gn = reinterpret_cast<const char*>(g) + ((t_begin + vnext * V) << esh);
#pragma unroll
            for (int s = 0; s < P; ++s) {
                if (s < theta) prefetch_l1(gn + (plan.woff[s] << esh));
            }
            if constexpr (PREAGG) {
                for (int k = 0; k < plan.nbase; ++k) prefetch_l1(gn + (plan.boff[k] << esh));
                if (plan.loose_in_smem) {
                    for (int k = 0; k < plan.nloose; ++k) prefetch_l1(gn + (plan.loff[k] << esh));
                }
            }
        }

        if constexpr (PREAGG) {
            float T[V];
#pragma unroll
            for (int v = 0; v < V; ++v) T[v] = 0.0f;
            // base rows: summed as they arrive, 8 loads in flight
            const int nbase = plan.nbase;
            for (int base = 0; base < nbase; base += 8) {
                float x[8][V];
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    if (base + k < nbase) {
                        load_grad<V>(g, t + plan.boff[base + k], dtype, x[k]);
                    } else {
#pragma unroll
                        for (int v = 0; v < V; ++v) x[k][v] = 0.0f;
                    }
                }
#pragma unroll
                for (int k = 0; k < 8; ++k) {
#pragma unroll
                    for (int v = 0; v < V; ++v) T[v] += x[k][v];
                }
            }
            // loose rows: parked in this thread's shared-memory column
            const int nloose = plan.nloose;
            const bool in_smem = plan.loose_in_smem != 0;
            if (in_smem) {
                for (int base = 0; base < nloose; base += 8) {
                    float x[8][V];
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        if (base + k < nloose) load_grad<V>(g, t + plan.loff[base + k], dtype, x[k]);
                    }
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        if (base + k < nloose) store_vec<V>(xcol + size_t(base + k) * stride, x[k]);
                    }
                }
            }
            float C[V];
#pragma unroll
            for (int v = 0; v < V; ++v) C[v] = 0.0f;
            int kadd = 0;
#pragma unroll
            for (int s = 0; s < P; ++s) {
                if (s < theta) {
                    if ((corr_mask >> s) & 1ull) {
                        const int src = plan.src[s];
                        if (src == GAR_SRC_ZERO) {
#pragma unroll
                            for (int v = 0; v < V; ++v) C[v] = 0.0f;
                        } else if (src != GAR_SRC_CONT) {
                            read_vec<V>(tcol + size_t(src) * stride, C);
                        }
                        const int kend = kadd + plan.nadd[s];
                        for (; kadd < kend; ++kadd) {
                            float x[V];
                            const int pos = plan.add_pos[kadd];
                            if (in_smem) read_vec<V>(xcol + size_t(pos) * stride, x);
                            else load_grad<V>(g, t + plan.loff[pos], dtype, x);
#pragma unroll
                            for (int v = 0; v < V; ++v) C[v] += x[v];
                        }
                        const int sv = plan.save[s];
                        if (sv != GAR_SAVE_NONE) store_vec<V>(tcol + size_t(sv) * stride, C);
                    }
                    if ((chain_mask >> s) & 1ull) {
#pragma unroll
                        for (int v = 0; v < V; ++v) T[v] += e[s][v];
                    }
                    const float im = plan.inv_m[s];
#pragma unroll
                    for (int v = 0; v < V; ++v) a[s][v] = (T[v] + C[v]) * im;
                } else {
#pragma unroll
                    for (int v = 0; v < V; ++v) a[s][v] = 0.0f;
                }
            }
        } else {
#pragma unroll
            for (int s = 0; s < P; ++s) {
#pragma unroll
                for (int v = 0; v < V; ++v) a[s][v] = e[s][v];
            }
        }

        float res[V];
        k3_finish<P, V>(e, a, theta, beta, inv_beta, lo_pads, PREAGG && med_agr, even_mean, median_only, res);
        k3_store<V>(out, t, res);
    }
}

template <int P, bool EXACT, bool PREAGG, int V>
__global__ void __launch_bounds__(K3_THREADS)
k3_coordinate(const float* __restrict__ g, int n, int theta_arg, int64_t t_begin, int64_t t_end, int64_t ld,
              gar_selection_t* __restrict__ sel, const K3Out out, int loose_cap, int dtype) {
    k3_coordinate_body<P, EXACT, PREAGG, V>(g, n, theta_arg, t_begin, t_end, ld, sel, out, loose_cap, dtype, blockIdx.x, gridDim.x);
}
// Batch mode: CTA b takes its tensor (gradients, output, d, row stride) from the descriptor
// multi[cta_desc[b]] and the selection sel + index * sel_stride.
template <int P, bool EXACT, bool PREAGG, int V>
__global__ void __launch_bounds__(K3_THREADS)
k3_coordinate_multi(const MultiDesc* __restrict__ multi, const int* __restrict__ cta_desc, int n, int theta_arg,
                    gar_selection_t* __restrict__ sel, int sel_stride, int loose_cap, float lr, float mu, int dtype) {
    const MultiDesc t = multi[cta_desc[blockIdx.x]];
    const K3Out out{t.out, t.x, t.v, lr, mu};
    k3_coordinate_body<P, EXACT, PREAGG, V>(static_cast<const float*>(t.grads), n, theta_arg, 0, t.d, t.ld,
                                            sel + size_t(t.index) * sel_stride, out, loose_cap, dtype,
                                            blockIdx.x - unsigned(t.cta_first), unsigned(t.ctas));
}

template <int P>
cudaError_t launch_k3_p(const float* g, int n, int64_t d, int64_t ld, gar_selection_t* sel, int theta, int preagg,
                        int vec, int bulk_ctas, const K3Out& out, int sm_count, cudaStream_t stream, int dtype);
template <int P> int bulk_ctas_for(int n, int theta, int preagg);
template <int P>
cudaError_t launch_k3_multi_p(const MultiDesc* desc, const int* cta_desc, int total_ctas, int n, int theta, int preagg, int vec,
                              gar_selection_t* sel, int sel_stride, float lr, float mu, int dtype, cudaStream_t stream);
template <int P> int k3_multi_threads(int n, int preagg, int vec);

}  // namespace gar
