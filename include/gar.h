/*
 * gar.h -- C ABI of the gradient aggregation rule (GAR) library for NVIDIA B200
 * (sm_100a): averaging, coordinate-wise median, Krum, multi-Krum, Bulyan and
 * multi-Bulyan of n worker gradients of dimension d, 1 <= n <= 64, fp32.
 *
 * The operations follow "Fast and Robust Distributed Learning in High
 * Dimension" (the multi-Bulyan paper): Eq. 4 and Algorithm 1 (functions
 * multi-Krum, multi-Bulyan and GAR), the one-sentence Bulyan of Section 2.2,
 * the averaging rule of the Introduction and the Median rule of Section 5.
 *
 * General conventions
 *  - "dev" pointers are device pointers of the current CUDA device, "host"
 *    pointers are host pointers.  All buffers are owned by the caller.
 *  - Gradients are row-major: worker i occupies grads[i*ld .. i*ld + d).
 *    Any alignment and any ld >= d are accepted; the vectorised kernels are
 *    used when grads and out are 16-byte aligned and ld is a multiple of 4.
 *  - Every call is asynchronous on `stream` (a cudaStream_t passed as void*;
 *    NULL is the legacy default stream) unless stated otherwise.  There is no
 *    host synchronisation and no host round trip between the kernels.
 *  - Argument and precondition errors are returned before anything is
 *    launched; launch failures are returned as GAR_ERR_CUDA.  No exceptions
 *    cross this boundary.  There is no CPU fallback.
 *  - Results are deterministic: the same input gives bit-identical output.
 *  - Ties (equal scores, equal distances to the median) are broken towards the
 *    lowest worker index, in the coordinate phase towards the earliest round.
 *    The median of an even count is the lower of the two middle values unless
 *    GAR_EVEN_MEDIAN_MEAN is asked for.  A non-finite distance is treated as
 *    +infinity.
 *  - No silent wrong answer: if a kernel gives up on one of its bounded waits, or
 *    the coordinate phase is handed an inconsistent selection, the selection's
 *    `status` is set and `out` is filled with NaN (see GAR_ERR_TIMEOUT below).
 *  - Thread safety: calls on distinct devices, or with distinct caller workspaces
 *    on distinct streams, may run concurrently.  The cached per-device buffers
 *    (NULL workspace, gar_aggregate_host, gar_pairwise_distances_static) are
 *    created under a lock but shared: serialise the calls that use them.
 *
 * Distances for 16 < n <= 64 (16-byte aligned rows, d >= 32768) are formed on the
 * tensor cores from rows rounded to a grid of 2^-21 of the largest binade each row
 * has shown; the kernel then bounds the effect of that rounding on every D_ij from
 * the steps it used (rounding errors taken as independent of the differences, six
 * standard deviations, plus the worst-case bias) and, if some pair's bound exceeds
 * 1e-6 of its distance, the same call recomputes the matrix with the fp32
 * difference form on the CUDA cores, on the device and without a host round trip
 * (about 2.5 times slower).  Inputs that stay on the fast path: rows whose largest
 * entry R and typical difference to the other rows s satisfy roughly
 * R / s <= 0.2 sqrt(d) (e.g. 100 at d = 2.6e5, 1000 at d = 2.6e7).  Rows that agree
 * within the grid everywhere are reported at distance exactly 0.
 */
#ifndef GAR_H_
#define GAR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define GAR_MAX_N 64
#define GAR_VERSION 105

typedef enum {
    GAR_AVERAGE      = 0, /* (1/n) sum_i G_i                       (Introduction)            */
    GAR_MEDIAN       = 1, /* coordinate-wise median                (Section 5, "Median")     */
    GAR_KRUM         = 2, /* smallest-score gradient               (Eq. 4 with m = 1)        */
    GAR_MULTI_KRUM   = 3, /* average of the m best-scored          (Eq. 4; Alg. 1 multi-Krum)*/
    GAR_BULYAN       = 4, /* theta = n-2f Krum winners, median, beta closest (Section 2.2;
                             iteration count of the proof of Theorem 2 (i))                  */
    GAR_MULTI_BULYAN = 5  /* Algorithm 1: theta = n-2f-2 rounds, pre-aggregated G^agr,
                             median of G^ext, beta = theta-2f closest entries of G^agr       */
} gar_rule_t;

typedef enum {
    GAR_OK               = 0,
    GAR_ERR_INVALID_ARG  = 1, /* null pointer, n < 1, f < 0, d < 1, ld < d, unknown rule, bad option */
    GAR_ERR_PRECONDITION = 2, /* n < 2f+3 (Krum family) or n < 4f+3 (Bulyan family), Section 2.2    */
    GAR_ERR_UNSUPPORTED  = 3, /* n > GAR_MAX_N                                                       */
    GAR_ERR_WORKSPACE    = 4, /* workspace missing, misaligned (256 B) or too small                  */
    GAR_ERR_CUDA         = 5, /* a CUDA runtime call or a launch failed                              */
    GAR_ERR_TIMEOUT      = 6  /* a bounded device-side wait gave up.  The asynchronous calls cannot
                                 return it; it travels on the device instead: a distance kernel that
                                 gives up fills the whole matrix, diagonal included, with NaN; the
                                 selection kernel answers a NaN diagonal with status = GAR_ERR_TIMEOUT
                                 and selects nothing; the coordinate kernel answers any status other
                                 than GAR_OK by filling `out` with NaN, and stores GAR_ERR_TIMEOUT
                                 itself if one of its own waits gives up.  gar_aggregate_host, which
                                 is synchronous, returns the status. */
} gar_status_t;

typedef enum {
    GAR_EVEN_MEDIAN_LOWER = 0, /* median of an even count = the lower middle value (what the Median
                                  comparator of Section 5, PyTorch's, returns)                      */
    GAR_EVEN_MEDIAN_MEAN  = 1  /* = the mean of the two middle values                               */
} gar_even_median_t;

typedef enum {
    GAR_F32  = 0, /* IEEE binary32 (the default everywhere)                                        */
    GAR_BF16 = 1, /* bfloat16 gradients: every value is widened to fp32 exactly as it is loaded   */
    GAR_F16  = 2  /* IEEE binary16 gradients, likewise; all arithmetic and the output stay fp32   */
} gar_dtype_t;

typedef enum {
    GAR_DISTANCES_AUTO       = 0, /* tensor-core Gram product where it applies, checked as described above */
    GAR_DISTANCES_DIFFERENCE = 1  /* always the fp32 difference form on the CUDA cores                     */
} gar_distance_mode_t;

/*
 * Result of the scoring / selection step (Eq. 4; Algorithm 1, multi-Krum and
 * the extraction loop of multi-Bulyan), device resident, consumed by the
 * coordinate phase.  Rounds are numbered 0..theta-1 in extraction order.
 *   winners[r]  index of the smallest-score gradient of round r (G^ext[r])
 *   sets[r]     bit i set <=> gradient i is averaged into G^agr[r]
 *   m[r]        number of bits in sets[r]
 *   scores[r][i] score of gradient i in round r (+inf if already extracted)
 *   gap_winner[r], gap_set[r]  relative gaps (s2-s1)/s2 between the two
 *               smallest scores and between the m-th and (m+1)-th score
 * The fields from `nu` on are the summation plan the coordinate kernel executes
 * for the pre-aggregating rules.  Rounds are visited last-to-first ("slots":
 * slot s = round theta-1-s); the sets lose about one gradient per round, so in
 * slot order they mostly grow.  With T_s the sum over slot s's set:
 *     T_s = sum(base rows) + sum(winners of the slots t <= s in chain_mask) + C_s
 *   base_rows[0..nbase)  gradients present in every slot (minus a chained slot-0 winner)
 *   chain_mask  bit s: the winner of slot s is in every set from slot s on; it is
 *               added to the running sum at slot s (the winner's value is needed
 *               there anyway)
 *   loose_rows[0..nloose)  every other gradient that occurs in some set
 *   C_s         sum over the loose gradients of slot s, built by a small plan:
 *               slot_src[s] says where it starts (GAR_SRC_ZERO, GAR_SRC_CONT =
 *               continue from slot s-1, or the index of a saved sum),
 *               slot_nadd[s] loose gradients are added (positions in loose_rows,
 *               consecutive in add_pos[], slot 0 first), slot_save[s] is
 *               GAR_SAVE_NONE or the index under which C_s is kept
 *   corr_mask   bit s: slot s has anything to do for C_s
 * Sums are only ever added to, never subtracted from.
 */
#define GAR_SRC_ZERO  255
#define GAR_SRC_CONT  254
#define GAR_SAVE_NONE 255
#define GAR_MAX_SAVED 8
typedef struct {
    int32_t  n, f, rule, theta, beta;
    int32_t  preagg;              /* 1: G^agr[r] = mean over sets[r]; 0: G^agr = G^ext */
    int32_t  median_of_agr;       /* 1: median taken over G^agr instead of G^ext       */
    int32_t  status;              /* gar_status_t written by the selection kernel (GAR_ERR_TIMEOUT if
                                     the distance matrix carries a NaN diagonal); the coordinate
                                     kernel stores GAR_ERR_TIMEOUT (a wait of its own gave up) or
                                     GAR_ERR_INVALID_ARG (tables inconsistent with its arguments)
                                     and fills `out` with NaN whenever this is not GAR_OK */
    int32_t  even_median;         /* gar_even_median_t */
    int32_t  reserved;
    int32_t  winners[GAR_MAX_N];
    int32_t  m[GAR_MAX_N];
    uint64_t sets[GAR_MAX_N];
    double   gap_winner[GAR_MAX_N];
    double   gap_set[GAR_MAX_N];
    /* summation plan */
    int32_t  nu;                  /* number of distinct gradients read                  */
    int32_t  total_adds;          /* sum of slot_nadd                                   */
    int32_t  nbase, nloose;
    uint64_t chain_mask, corr_mask;
    uint8_t  base_rows[GAR_MAX_N];
    uint8_t  loose_rows[GAR_MAX_N];
    uint8_t  slot_src[GAR_MAX_N];
    uint8_t  slot_save[GAR_MAX_N];
    uint8_t  slot_nadd[GAR_MAX_N];
    uint8_t  add_pos[GAR_MAX_N * GAR_MAX_N];
    double   scores[GAR_MAX_N][GAR_MAX_N];
} gar_selection_t;

/* Extended call.  Zero-initialise, then set what you need. */
typedef struct {
    int32_t       rule;           /* gar_rule_t */
    int32_t       n, f;
    int64_t       d;
    int64_t       ld;             /* row stride in elements; 0 means d */
    const float*  grads;          /* dev, n rows */
    float*        out;            /* dev, d values; must not overlap grads (may be NULL with sgd_params) */
    void*         stream;         /* cudaStream_t */
    void*         workspace;      /* dev, 256-byte aligned, >= gar_workspace_bytes(), its first 256
                                     bytes zeroed once before the first use (the kernels restore
                                     them); NULL: the library's cached per-device workspace
                                     (allocated on first use) */
    size_t        workspace_bytes;
    int32_t       m;              /* multi-Krum only: number of averaged gradients, 1..n-f-2; 0 = n-f-2
                                     (Section 3 allows any m <= n-f-2) */
    int32_t       theta;          /* multi-Bulyan only: number of rounds, 2f+1..n-2f-2; 0 = n-2f-2 */
    int32_t       median_of_agr;  /* multi-Bulyan only: 1 = median over G^agr (reading of Section 5.2's
                                     "median ... over ... pre-aggregated gradients"); 0 = Algorithm 1 */
    int32_t       even_median;    /* gar_even_median_t: median of an even count (Median rule of Section 5;
                                     Median(G^ext) of Algorithm 1 when theta is even) */
    double*       dist_out;       /* optional dev [n*n]: the distance matrix */
    gar_selection_t* selection_out; /* optional dev: the selection result */
    int32_t       distance_mode;  /* gar_distance_mode_t */
    int32_t       grads_dtype;    /* gar_dtype_t of `grads` (ld counts elements of that type).  16-bit
                                     gradients halve the bytes both passes read; every value is widened to
                                     fp32 exactly where it is loaded, all arithmetic and the output stay
                                     fp32.  Supported by gar_aggregate_ex only (the stage calls take fp32).
                                     The staged kernels need 16-byte aligned rows (ld a multiple of 8). */
    /* Optional SGD step fused into the coordinate kernel's store (Eq. 2: x <- x - lr * GAR(...);
       Section 5.1 trains with momentum 0.9): with g the aggregated coordinate,
           v <- sgd_momentum * v + g   (only if sgd_momentum_buf is given),   x <- x - sgd_lr * v   (or g)
       so the aggregate never makes a round trip through memory.  sgd_params NULL: no step.
       With a step, `out` may be NULL (the aggregate itself is then not stored).  If the call ends
       with a status other than GAR_OK in the selection, x and v are left untouched. */
    float*        sgd_params;       /* dev [d], x, updated in place */
    float*        sgd_momentum_buf; /* dev [d], v, updated in place; NULL: plain SGD */
    float         sgd_lr;
    float         sgd_momentum;
} gar_params_t;

/* Library version (GAR_VERSION).  The paper has no counterpart. */
int gar_version(void);

/* Static description of a status code. */
const char* gar_status_string(int status);

/* The CUDA runtime error (a cudaError_t value; 0 = none yet) behind the calling thread's latest
 * GAR_ERR_CUDA return, and the runtime's own name for it (a static string; "cudaSuccess" when
 * there was none).  Kept per host thread; a later successful call does not clear it.  The paper
 * has no counterpart. */
int gar_last_cuda_error(void);
const char* gar_last_cuda_error_name(void);

/* theta (number of extraction rounds) and beta (values kept per coordinate) of a
 * rule: multi-Bulyan n-2f-2 and theta-2f (Algorithm 1); Bulyan n-2f and theta-2f
 * (Section 2.2 / proof of Theorem 2); Krum, multi-Krum, averaging 1 and 1;
 * median n and 1.  Returns -1 if the rule's precondition fails. */
int gar_theta(int rule, int n, int f);
int gar_beta(int rule, int n, int f);

/* Bytes of device workspace a call needs (host, pure).  0 on invalid arguments.
 * The first 256 bytes are a control block of 32-bit words: [0] ticket counter of the distance
 * kernels (zero between calls), [2] set to 1 by a distance kernel whose wait gave up, [4] how the
 * last distance call ran: 0 = fp32 difference form, 1 = tensor-core Gram product kept,
 * 2 = Gram product rejected by its error bound and recomputed in the difference form. */
size_t gar_workspace_bytes(int rule, int n, int f, int64_t d);

/*
 * GAR(f, [G_1..G_n]) of Algorithm 1 for the chosen rule.
 *   grads dev [n rows, stride d], out dev [d].
 * Uses a per-device workspace that the library allocates on the first call for
 * that device and keeps until gar_shutdown().  Not re-entrant across streams
 * for the same device (the cached workspace is shared); use gar_aggregate_ex
 * with distinct workspaces for concurrent calls.
 */
int gar_aggregate(int rule, const float* grads, int n, int f, int64_t d, float* out, void* stream);

/* Same with explicit row stride, caller workspace, options and optional outputs. */
int gar_aggregate_ex(const gar_params_t* params);

/*
 * The same rule on HOST buffers: grads host [n rows, stride d], out host [d].
 * Copies the rows to a device buffer the library caches (grown on demand, kept
 * until gar_shutdown), runs the three kernels and copies the result back, all
 * on one internal stream.  Synchronous: returns when `out` is complete.
 * Pinned (page-locked) host buffers are copied at full PCIe speed; pageable
 * ones work but are slower.
 */
int gar_aggregate_host(int rule, const float* grads, int n, int f, int64_t d, float* out);

/*
 * Step 1 alone: D_ij = ||G_i - G_j||^2 (Algorithm 1, multi-Krum, neighbour
 * distances), all pairs, one streaming pass.  dist dev [n*n] fp64, symmetric,
 * zero diagonal.  workspace as in gar_params_t (NULL = cached).
 */
int gar_pairwise_distances(const float* grads, int n, int64_t d, int64_t ld, double* dist,
                           void* workspace, size_t workspace_bytes, void* stream);
/* Same with a gar_distance_mode_t. */
int gar_pairwise_distances_mode(const float* grads, int n, int64_t d, int64_t ld, double* dist,
                                void* workspace, size_t workspace_bytes, int distance_mode, void* stream);

/*
 * Sum of `count` distance matrices in the order given: dist = parts[0] + parts[1] + ... (fp64,
 * element by element, left to right).  This is the one exchange step of an aggregation whose
 * coordinates are sharded over several GPUs (the dimension d of the Introduction's footnote,
 * 10^9 to 10^11, does not fit one device; Theorem 2 (ii): the work is O(d) and splits along d):
 * every GPU computes gar_pairwise_distances on its own slice of the columns -- squared distances
 * add over disjoint column sets -- the n*n partial matrices are all-gathered into every GPU's own
 * memory, and each GPU adds them in rank order with this call, so that all of them hold the
 * bit-identical matrix, select the same gradients (gar_select) and run gar_coordinate_phase on
 * their own slice.  A NaN diagonal (a distance kernel that gave up) survives the sum.
 *   parts dev [count][n*n] fp64, dist dev [n*n] (may be parts[0]); 1 <= count <= 1024.
 */
int gar_reduce_partials(const double* parts, int count, int n, double* dist, void* stream);

/*
 * Many small tensors in one launch sequence.  A model's gradient usually sits in memory as one
 * tensor per layer; aggregating those one call at a time costs three kernel launches per tensor,
 * which dominates below about 10^6 coordinates.  This call takes `count` tensors that share rule,
 * n and f -- tensor t is an n x d[t] block of gradients, row i from worker i -- and runs each
 * stage once over all of them: three to seven launches whatever the count (tensors whose addresses
 * allow wide accesses and those that do not are launched separately).  The gradients are fp32,
 * or bfloat16 / binary16 for all tensors alike (grads_dtype), widened exactly as they are loaded.
 *   joint = 0: every tensor is a problem of its own: own distance matrix, own selection, own
 *              coordinate phase (Algorithm 1 applied per tensor; the paper has no counterpart).
 *   joint = 1: the tensors are the pieces of ONE gradient in R^d, d = sum of d[t] (Section 2.1: the
 *              rule acts on the whole gradient): the per-tensor distance matrices are added in the
 *              order given (squared distances add over disjoint coordinates), one selection is
 *              made, and every tensor's coordinate phase uses it.  The result equals
 *              gar_aggregate on the concatenation up to the summation order of the distances.
 * Distances use the fp32 difference form (Eq. 4's ||G_i - G_j||^2 term by term).  The work is
 * split over CTAs in proportion to the tensors' lengths, so a few long tensors among many short
 * ones are fine, but a batch of long tensors (above about 10^7 coordinates each) is served better
 * by one gar_aggregate_ex per tensor.
 *   tensors    HOST array of `count` entries, read before the call returns; grads / out device
 *              pointers, ld = 0 means d; no output (out, sgd_params, sgd_momentum_buf) may
 *              overlap any tensor's gradients or another output.
 *   workspace  device, 256-byte aligned, >= gar_multi_workspace_bytes(rule, n, f, count); it may
 *              hold anything on entry and must not be shared by calls in flight on other streams.
 *   dist_out   optional, device: joint ? n*n : count*n*n doubles (tensor t's matrix at t*n*n).
 *   selection_out  optional, device: joint ? 1 : count entries; its status field reports a
 *              selection that could not be made (the outputs are then NaN), as for gar_aggregate_ex.
 * Returns GAR_OK once everything is enqueued on `stream`.  The call copies a table it builds from
 * `tensors` out of a temporary host buffer, so it must not be recorded into a CUDA graph; calls
 * from several host threads are fine as long as each uses its own workspace.
 */
typedef struct gar_tensor_t {
    const void*  grads;            /* fp32, or 16-bit elements by gar_multi_params_t.grads_dtype */
    float*       out;              /* d values; may be NULL when sgd_params is given */
    int64_t      d;
    int64_t      ld;
    /* Optional SGD step fused into the store of this tensor's aggregate g (Eq. 2), as in
       gar_params_t, with the step size and momentum of gar_multi_params_t:
           v <- sgd_momentum * v + g   (only if sgd_momentum_buf is given),   x <- x - sgd_lr * v   (or g) */
    float*       sgd_params;       /* dev [d], x, updated in place; NULL: no step */
    float*       sgd_momentum_buf; /* dev [d], v, updated in place; NULL: plain SGD */
} gar_tensor_t;

typedef struct gar_multi_params_t {
    int32_t  rule, n, f, count;
    int32_t  joint;
    int32_t  even_median;            /* gar_even_median_t */
    const gar_tensor_t* tensors;
    void*    workspace;
    size_t   workspace_bytes;
    double*  dist_out;
    gar_selection_t* selection_out;
    void*    stream;
    float    sgd_lr;
    float    sgd_momentum;
    int32_t  grads_dtype;            /* gar_dtype_t: element type of every tensor's gradients (d, ld in elements) */
} gar_multi_params_t;

size_t gar_multi_workspace_bytes(int rule, int n, int f, int count);
int gar_aggregate_multi(const gar_multi_params_t* params);

/*
 * Step 1 alone, for callers that must not allocate: the same distance kernels, but
 * their scratch (ticket counter and per-CTA partial sums) is a fixed array inside the
 * library image instead of a workspace, so this call performs no cudaMalloc / cudaFree
 * and no other allocating call.  Meant for code that runs where device allocation is
 * impossible or unwanted: inside another framework's memory pool or a fixed memory
 * budget, with all of HBM already handed out, or in a latency-critical loop where an
 * allocation could synchronise the device.  The paper has no counterpart.
 *   - The array is about 10.9 MB (256 B + 592 CTAs x 2304 sums x 8 B) and is held by every
 *     GPU that loads the library until the process exits.  It covers every n <= GAR_MAX_N
 *     and any d; n > GAR_MAX_N returns GAR_ERR_UNSUPPORTED.
 *   - The first call on a device looks up the array's device address; make that first call
 *     before any stream capture.
 *   - All calls on a device share the array.  Each call clears the counter it needs on
 *     `stream` first, but two calls that overlap on the GPU (different streams) race:
 *     serialise them.
 *   grads dev [n rows, stride ld (0 = d)], dist dev [n*n] fp64; asynchronous on `stream`.
 */
int gar_pairwise_distances_static(const float* grads, int n, int64_t d, int64_t ld, double* dist,
                                  void* stream);

/*
 * Step 2 alone: scoring and iterative selection from a distance matrix
 * (Eq. 4; Algorithm 1 multi-Krum and the loop of multi-Bulyan).
 *   dist dev [n*n] fp64; sel dev, written.  m, theta, median_of_agr, even_median as in
 *   gar_params_t (0 = default).  A NaN on the diagonal of dist (left by a distance kernel
 *   that gave up) gives sel->status = GAR_ERR_TIMEOUT and no selection.
 */
int gar_select(int rule, const double* dist, int n, int f, int m, int theta, int median_of_agr,
               int even_median, gar_selection_t* sel, void* stream);

/*
 * Builds the coordinate kernel's schedule for GIVEN winners and sets (e.g. the
 * oracle's), without scoring: sel dev with n, f, rule, theta, beta, preagg,
 * median_of_agr, winners, sets filled by the caller; m and the summation plan
 * (nu .. add_pos) are written.  The paper has no counterpart
 * (test and diagnostic aid).
 */
int gar_schedule_from_tables(gar_selection_t* sel, void* stream);

/*
 * Step 3 alone: the coordinate phase (Algorithm 1, multi-Bulyan: Median of
 * G^ext, the beta entries of G^agr closest to it, their average) for a
 * selection already on the device.  theta and preagg repeat sel->theta and
 * sel->preagg (the host needs them to pick the kernel).  out dev [d].
 * Before it reads a gradient the kernel checks the selection on the device: a
 * status other than GAR_OK, a theta or preagg that differs from sel's, or a row
 * index >= n in the tables gives out = NaN everywhere (and, for the last two,
 * sel->status = GAR_ERR_INVALID_ARG); sel is therefore not const.
 */
int gar_coordinate_phase(const float* grads, int n, int64_t d, int64_t ld,
                         gar_selection_t* sel, int theta, int preagg, float* out, void* stream);

/*
 * Self-test of the bounded wait every staged kernel uses (mbarrier.try_wait in a loop with an
 * iteration limit): one warp waits, with the given limit (1 .. 65536), on a barrier that nothing
 * ever arrives on -- no copy and no tensor-core operation is in flight -- and reports how it
 * ended.  result dev [2] int64: [0] = GAR_ERR_TIMEOUT if the wait gave up as it must (GAR_OK
 * would mean it returned as if the barrier had completed), [1] = nanoseconds the wait took
 * (%globaltimer).  On B200 one suspended poll takes 4.0 microseconds; the kernels' own limit
 * is 2^20 polls, about 4.2 seconds.  The paper has no counterpart (diagnostic aid).
 */
int gar_selftest_bounded_wait(unsigned int limit, long long* result, void* stream);

/* Frees every cached device buffer of every device.  Synchronises. */
void gar_shutdown(void);

#ifdef __cplusplus
}
#endif
#endif /* GAR_H_ */
