/*
 * lsgd.h — C ABI of liblsgd: the data-parallel hot path of one round of
 * system-aware biased local SGD on a single NVIDIA B200 (sm_100a).
 *
 * The path has three parts (paper: Algorithm 1, Section 4.2, Section 4.3):
 *   1. the per-sample loss record  — a softmax cross-entropy scorer that turns a
 *      candidate pool's logits and labels into one loss per sample;
 *   2. the deterministic loss-based top-k selection for the fast workers;
 *   3. the biased model aggregation x_{t+1} = sum_i w_i * x^i_t   (Eq. 3).
 *
 * Conventions shared by every entry point
 *   - "device" pointers are CUDA global-memory addresses on the CURRENT device;
 *     "host" pointers are ordinary process memory.  Each argument says which.
 *   - The caller owns every buffer, including the workspace.  The library
 *     allocates no device memory, frees nothing and keeps no pointer after the
 *     kernels it enqueued have run.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *     stream).  Calls only enqueue work on that stream and return; they do not
 *     synchronise, except lsgd_read_device_status.
 *   - Errors are reported by return value only.  Argument errors are found on
 *     the host before anything is launched, so a failing call has no effect on
 *     the device.  No kernel traps.  One kernel has thread blocks that wait for
 *     each other: the selector for pools above 65,536 entries, launched
 *     cooperatively (all its blocks resident at once) with a barrier whose polls
 *     are counted; if the count ever ran out the kernel would give up, leave its
 *     outputs unspecified and record LSGD_ERR_TIMEOUT in the status block.
 *   - A size of zero (N == 0, k == 0, D == 0) is legal: the call returns LSGD_OK
 *     without launching anything.
 *   - Workspaces must be 256-byte aligned.  Their contents are scratch: they
 *     need no initialisation and have no meaning after the call, except for the
 *     status block read by lsgd_read_device_status.
 *   - Two calls that use the same workspace must be ordered on one stream.
 */
#ifndef LSGD_H_
#define LSGD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(_WIN32)
#define LSGD_API
#else
#define LSGD_API __attribute__((visibility("default")))
#endif

typedef enum lsgd_status {
    LSGD_OK = 0,
    LSGD_ERR_INVALID_ARG = 1, /* NULL where data is needed, negative size, k > N, P out of range, overlap */
    LSGD_ERR_UNSUPPORTED = 2, /* a dtype / order value the library does not know, N >= 2^31          */
    LSGD_ERR_ALIGNMENT = 3,   /* pointer not aligned to its element size, workspace not to 256 B      */
    LSGD_ERR_WORKSPACE = 4,   /* ws_bytes smaller than the matching *_workspace_bytes query           */
    LSGD_ERR_CUDA = 5,        /* the CUDA runtime refused a launch                                    */
    LSGD_ERR_TIMEOUT = 6      /* a bounded device-side wait ran out (reported by lsgd_read_device_status)       */
} lsgd_status;

/* Element type of the logits. Labels are always int64, losses always fp32. */
typedef enum lsgd_dtype { LSGD_F32 = 0, LSGD_BF16 = 1 } lsgd_dtype;

/* Order of the k selected indices.  Both orders are unique for a given input. */
typedef enum lsgd_order {
    LSGD_ORDER_LOSS_DESC = 0, /* highest loss first; equal losses by ascending index */
    LSGD_ORDER_INDEX_ASC = 1  /* the same set, ascending index                       */
} lsgd_order;

/* Largest number of worker replicas one lsgd_aggregate call accepts. */
#define LSGD_MAX_REPLICAS 64

/* Library version as major*10000 + minor*100 + patch. */
LSGD_API int lsgd_version(void);

/* Static, NUL-terminated description of a status code (never NULL). */
LSGD_API const char* lsgd_status_string(int status);

/* ------------------------------------------------------------------------- */
/* Workspace sizes (host-only arithmetic; 0 on invalid arguments).            */
/* ------------------------------------------------------------------------- */
LSGD_API size_t lsgd_score_workspace_bytes(int64_t N, int64_t T, int64_t C);
LSGD_API size_t lsgd_topk_workspace_bytes(int64_t N, int64_t k);
LSGD_API size_t lsgd_score_topk_workspace_bytes(int64_t N, int64_t T, int64_t C, int64_t k);

/*
 * lsgd_score_losses — the per-sample loss record of Algorithm 1 (the step of
 * the training loop that stores the loss of every processed sample; one float
 * per sample, as Section 4.4 "Potential Limitations" counts it).  The loss
 * f(x, xi) of the problem definition (Section 2) is taken to be softmax
 * cross-entropy with natural log.
 *
 *   token loss   l[n,t] = -log softmax(logits[n,t,:])[labels[n,t]]
 *   sample loss  losses[n] = mean of l[n,t] over the tokens t whose label is not
 *                ignore_index, summed in a fixed order; 0 if every token of the
 *                sample is ignored.  T == 1 is plain classification.
 *
 *   logits  device, [N, T, C] row-major, contiguous, dtype `dtype`, aligned to
 *           its element size (16-byte alignment is faster, not required).
 *           Values must be finite with |x| <= 1e8: the kernels work with
 *           x * log2(e) rounded to fp32 and carry the rounding error of that
 *           product for the row maximum along exactly, which needs it to stay
 *           within the range of an exponent (it is at most 8 for |x| <= 1e8);
 *           beyond that range results are unspecified.  Rows whose label is
 *           ignore_index are not scored,
 *           and rows longer than 2 KB are then not read at all (shorter rows are
 *           loaded in contiguous tiles, ignored rows included; their values are
 *           not used).
 *   labels  device, [N, T] int64.  A label outside [0, C) that is not
 *           ignore_index makes that token's loss NaN (and so the sample's) and
 *           is counted in the status block.
 *   losses  device, [N] fp32, written in full.  Must not overlap logits.
 *   ws      device workspace of at least lsgd_score_workspace_bytes(N, T, C).
 *
 * Arithmetic is fp32 (bf16 logits are widened exactly); results are within
 * 1e-5 relative of an exact evaluation, also for losses near zero.
 * Results do not depend on the launch geometry: same input, same bits.
 */
LSGD_API lsgd_status lsgd_score_losses(const void* logits, lsgd_dtype dtype, const int64_t* labels,
                                       int64_t N, int64_t T, int64_t C, int64_t ignore_index,
                                       float* losses, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * lsgd_topk_select — deterministic loss-based top-k selection (Section 4.2,
 * "Data Allocation for Fast Workers"; Algorithm 1, the step that picks the
 * highest-loss samples).  Selects the k entries that come first in the total order
 *     higher loss first, then lower index,
 * where -0.0 equals +0.0 and every NaN ranks above +inf (NaNs tie with each
 * other).  Exact: integer comparisons only, bit-reproducible.
 *
 *   losses    device, [N] fp32.  N < 2^31: indices are 32-bit, as the index
 *             payload quoted in Section 4.2 implies.
 *   k         0 <= k <= N.
 *   out_idx   device, [k] int32, the selected indices in `order`.
 *   out_vals  device, [k] fp32 or NULL: losses[out_idx[j]], bits unchanged.
 *   ws        device workspace of at least lsgd_topk_workspace_bytes(N, k).
 * One kernel per call: pools of up to 1,024 entries in one thread block, up to
 * 65,536 in one thread-block cluster, larger ones in a cooperative launch.
 */
LSGD_API lsgd_status lsgd_topk_select(const float* losses, int64_t N, int64_t k, lsgd_order order,
                                      int32_t* out_idx, float* out_vals, void* ws, size_t ws_bytes,
                                      void* cuda_stream);

/*
 * lsgd_topk_select_static — lsgd_topk_select without a workspace argument, for
 * callers that cannot allocate device memory: code on a path where cudaMalloc
 * is not allowed (it synchronises the device and can fail late), programs whose
 * device memory is all owned by another framework's pool, or hosts with no
 * device allocator of their own.  The paper has no counterpart to this entry
 * point; it is a convenience of this library.
 *
 * The scratch is a fixed array of about 4.5 MiB inside the library's device
 * image (every GPU that loads the library holds it until the process ends), so
 * the pool is limited to N <= LSGD_STATIC_TOPK_MAX_N; a larger N returns
 * LSGD_ERR_UNSUPPORTED and nothing is launched.  Arguments, result and order are
 * exactly those of lsgd_topk_select.  The call allocates and frees nothing.
 *
 *   - The first call on each device looks up the array's device address
 *     (cudaGetSymbolAddress, with that device current).  Make that first call
 *     outside any stream capture.
 *   - All calls on a device share the one array, and it keeps the previous
 *     call's contents; the call clears what has to start at zero.  Two calls that
 *     can overlap on the GPU (different streams without an ordering between
 *     them) race on it: keep calls to this entry point on one stream, or order
 *     them with events.  lsgd_read_device_status does not apply to it.
 */
#define LSGD_STATIC_TOPK_MAX_N 262144
LSGD_API lsgd_status lsgd_topk_select_static(const float* losses, int64_t N, int64_t k, lsgd_order order,
                                             int32_t* out_idx, float* out_vals, void* cuda_stream);

/*
 * lsgd_score_topk — lsgd_score_losses followed by lsgd_topk_select on its
 * result, enqueued as one sequence in which the scorer's epilogue already
 * builds the selector's first radix histogram.  `losses` ([N], device) is
 * still written in full: it is the method's loss table.  Arguments as in the
 * two calls above; ws >= lsgd_score_topk_workspace_bytes(N, T, C, k).
 * Bit-identical to calling the two entry points one after the other.
 */
LSGD_API lsgd_status lsgd_score_topk(const void* logits, lsgd_dtype dtype, const int64_t* labels,
                                     int64_t N, int64_t T, int64_t C, int64_t ignore_index, int64_t k,
                                     lsgd_order order, float* losses, int32_t* out_idx, float* out_vals,
                                     void* ws, size_t ws_bytes, void* cuda_stream);

/* ------------------------------------------------------------------------- */
/* Per-epoch data allocation (Section 4.2, "Bias Injection via Data Sampling"; */
/* Algorithm 1, the four steps before the training loop).                      */
/* ------------------------------------------------------------------------- */
/*
 * Which calls make which allocation scheme (Section 4.2 and the appendix,
 * "Random Sampling Scheme Comparison" with its table of data sampling methods).
 * The library has no mode switch: a scheme is a choice of sizes and exclusion
 * lists by the caller.
 *   high-loss samples to the FAST group (the paper's method):
 *     fast list  = lsgd_fast_allocation(k_high = floor(lambda N_F), n_fill = N_F - k_high)
 *     slow list  = lsgd_draw_uniform(n_draw = N_S) on another stream   (separated sampling)
 *               or lsgd_draw_uniform(n_draw = N_S, exclude = fast list) (unified sampling:
 *                  the two lists then partition the N samples)
 *   high-loss samples to the SLOW group (the table's other row):
 *     slow list  = lsgd_fast_allocation(k_high = floor(lambda N_S), n_fill = N_S - k_high)
 *     fast list  = lsgd_draw_uniform(n_draw = N_F), with or without the slow list excluded
 *   unbiased baseline: lsgd_draw_uniform for both groups.
 * Each list is then cut into per-worker shares with lsgd_worker_share.
 */

/*
 * lsgd_allocation_sizes — how many of the N samples of an epoch each worker
 * group gets (Section 4.2): with P_F fast workers doing tau_F local steps per
 * round and P_S slow workers doing tau_S,
 *     N_F = floor(N * tau_F P_F / (tau_F P_F + tau_S P_S)),   N_S = N - N_F,
 *     k   = floor(lambda * N_F)      (the high-loss part of the fast allocation),
 * N_F in exact integer arithmetic; k from the product lambda * N_F in double,
 * where a product within 2^-51 (relative) below an integer counts as that
 * integer, so that a decimal lambda gives the decimal result (0.29 * 100 is
 * 28.999999999999996 in double; k = 29).  The paper gives the ratios
 * only; rounding N_F down and giving the slow workers the rest keeps one epoch
 * at N samples.  Host only.  tau and P values >= 0 with tau_F P_F + tau_S P_S > 0
 * and 0 <= lambda <= 1, else LSGD_ERR_INVALID_ARG.
 *   n_fast, n_slow, k_high   host, out
 */
LSGD_API lsgd_status lsgd_allocation_sizes(int64_t N, int32_t tau_fast, int32_t p_fast, int32_t tau_slow,
                                           int32_t p_slow, double lambda, int64_t* n_fast, int64_t* n_slow,
                                           int64_t* k_high);

/*
 * lsgd_worker_share — the even split of a list of n sample indices over the
 * P workers of a group (Section 4.2; Algorithm 1): worker p gets the contiguous
 * entries [begin, end) = [floor(p n / P), floor((p + 1) n / P)).  Shares differ
 * by at most one entry and cover the list exactly once.  Host only.
 */
LSGD_API lsgd_status lsgd_worker_share(int64_t n, int32_t P, int32_t p, int64_t* begin, int64_t* end);

/*
 * lsgd_draw_uniform — n_draw samples drawn uniformly at random, without
 * replacement, from the samples 0..N-1 that are not listed in exclude_idx
 * (Section 4.2, "Data Allocation for Slow Workers": the slow group's N_S samples
 * are such a draw from all N samples; with an exclusion list it is a draw from
 * the remaining samples, e.g. the unified-sampling variant of the appendix in
 * which the slow workers draw from what the fast workers left).
 *
 * Every sample i gets the random priority q_i = top 30 bits of word (i mod 4)
 * of the Philox4x32-10 block with counter (i div 4, 0, stream_lo, stream_hi) and
 * key (seed_lo, seed_hi).  The draw is the n_draw candidates that come first in
 * the order "higher q first, then lower index", written in that order: every
 * subset is equally likely and the order is a uniform random order (up to ties
 * among 30-bit priorities).  The same (N, seed, stream, exclusion) always gives
 * the same result; different `stream` values give independent draws, so a
 * caller can use e.g. stream = 2 * epoch for the fast group and 2 * epoch + 1
 * for the slow group (the paper's separated sampling).
 *
 *   exclude_idx  device, [n_exclude] int32 or NULL: distinct indices in [0, N)
 *                (entries outside that range are ignored).
 *   n_draw       0 <= n_draw <= N - n_exclude.
 *   out_idx      device, [n_draw] int32.  May not overlap exclude_idx.
 *   ws           device workspace of at least lsgd_draw_workspace_bytes(N, n_draw).
 */
LSGD_API size_t lsgd_draw_workspace_bytes(int64_t N, int64_t n_draw);
LSGD_API lsgd_status lsgd_draw_uniform(int64_t N, int64_t n_draw, uint64_t seed, uint64_t stream,
                                       const int32_t* exclude_idx, int64_t n_exclude, int32_t* out_idx, void* ws,
                                       size_t ws_bytes, void* cuda_stream);

/*
 * lsgd_fast_allocation — the fast workers' samples for one epoch (Section 4.2,
 * "Data Allocation for Fast Workers"; Algorithm 1: the highest-loss samples
 * first, then the rest of the allocation drawn at random from the samples that
 * were not selected):
 *     out_idx[0 .. k_high)               the k_high highest-loss samples, as
 *                                        lsgd_topk_select gives them in
 *                                        LSGD_ORDER_LOSS_DESC;
 *     out_idx[k_high .. k_high + n_fill) n_fill samples drawn as by
 *                                        lsgd_draw_uniform(seed, stream) with the
 *                                        first part as the exclusion list.
 * The list is then split over the fast workers with lsgd_worker_share.
 *
 *   losses   device, [N] fp32 (the loss table lsgd_score_losses writes).
 *   k_high + n_fill <= N.      out_idx  device, [k_high + n_fill] int32.
 *   ws       device workspace of at least
 *            lsgd_fast_allocation_workspace_bytes(N, k_high, n_fill).
 */
LSGD_API size_t lsgd_fast_allocation_workspace_bytes(int64_t N, int64_t k_high, int64_t n_fill);
LSGD_API lsgd_status lsgd_fast_allocation(const float* losses, int64_t N, int64_t k_high, int64_t n_fill,
                                          uint64_t seed, uint64_t stream, int32_t* out_idx, void* ws,
                                          size_t ws_bytes, void* cuda_stream);

/*
 * lsgd_aggregate — biased model aggregation, Eq. 3:  out[j] = sum_i w_i * x_i[j]
 * over the P worker replicas' flattened parameters, accumulated in fp32 in
 * ascending i (one multiply, then fused multiply-adds).  Every replica element
 * is read exactly once.
 *
 *   replicas  HOST array of P DEVICE pointers, each to D fp32 values, 4-byte
 *             aligned (16-byte alignment of all P pointers and of `out` takes
 *             the vectorised path).  Read before the call returns.
 *   weights   HOST array of P fp32 weights, read before the call returns, used
 *             exactly as given: not normalised, not clamped (Remark 2: any
 *             weight vector is admissible).  w_i == 0 does not skip replica i
 *             (IEEE rules: 0 * inf = NaN).
 *   P         1 <= P <= LSGD_MAX_REPLICAS.      D >= 0.
 *   out       device, [D] fp32.  May be exactly one of the replicas (in-place
 *             update); any other overlap with a replica is LSGD_ERR_INVALID_ARG.
 */
LSGD_API lsgd_status lsgd_aggregate(const float* const* replicas, const float* weights, int32_t P,
                                    int64_t D, float* out, void* cuda_stream);

/*
 * lsgd_aggregate_round — the aggregation step as one round of the training loop
 * needs it (Eq. 3; the local-SGD update rule of Section 2; Algorithm 1: after
 * the aggregation step every worker continues from x_{t+1}):
 *
 *   base == NULL:  x_{t+1}[j] = sum_i w_i x_i[j]                         (Eq. 3)
 *   base != NULL:  x_{t+1}[j] = base[j] + sum_i w_i (x_i[j] - base[j])   (Eq. 3 written around base = x_t, the
 *                  form of Section 2's rule, the previous model minus the averaged local progress; identical to Eq. 3 when the
 *                  weights sum to one, and more accurate in fp32 because the differences are small)
 *
 * accumulated in fp32 in ascending i (differences first, one multiply, fused multiply-adds, the base added last).
 * The result is written to `out` (fp32) and, if `broadcast` is non-zero, also into every replica, rounded to the
 * replicas' type (bf16: round to nearest even), all in the one pass that reads them.
 *
 *   replicas   HOST array of P DEVICE pointers, each to D values of type `dtype` (LSGD_F32 or LSGD_BF16), aligned
 *              to the element size (16-byte alignment of every pointer takes the vectorised path).  Read before the
 *              call returns.  Overwritten on the device when broadcast != 0.
 *   weights    HOST, P fp32, used as given (not normalised).      1 <= P <= LSGD_MAX_REPLICAS,  D >= 0.
 *   base       device, [D] fp32, or NULL.
 *   out        device, [D] fp32, or NULL when broadcast != 0 (the replicas then hold the result).
 *   Aliasing: `out` may be exactly `base`, and for fp32 replicas `out` or `base` may be exactly one replica; any
 *   partial overlap, and with broadcast any overlap between two replicas, is LSGD_ERR_INVALID_ARG.
 */
LSGD_API lsgd_status lsgd_aggregate_round(void* const* replicas, lsgd_dtype dtype, const float* weights, int32_t P,
                                          int64_t D, const float* base, float* out, int32_t broadcast,
                                          void* cuda_stream);

/*
 * lsgd_weights_from_steps — the weights of Eq. 3, w_i = tau_i / sum_j tau_j, from
 * the local step counts tau_i of the P workers.  Host only; computed in double
 * and rounded once to fp32.  tau_i >= 0 and sum > 0, else LSGD_ERR_INVALID_ARG.
 *   tau    host, [P] int32        w_out  host, [P] fp32
 */
LSGD_API lsgd_status lsgd_weights_from_steps(const int32_t* tau, int32_t P, float* w_out);

/*
 * lsgd_read_device_status — reads the status block that the last scoring or
 * selection call left at the start of `ws`.  Synchronises `cuda_stream`.
 *   bad_label_count  host, out: tokens whose label was outside [0, C) and not
 *                    ignore_index in that call.
 * Returns LSGD_ERR_CUDA if the copy failed, LSGD_ERR_TIMEOUT if the selector's barrier
 * gave up in that call (its outputs are then unspecified), else LSGD_OK.
 */
LSGD_API lsgd_status lsgd_read_device_status(const void* ws, int32_t* bad_label_count, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* LSGD_H_ */
