/*
 * abs_normtest.h -- C ABI of the norm-test + AdamW step for adaptive batch-size
 * training ("Adaptive Batch Size Schedules for Distributed Training of Language
 * Models with Data and Model Parallelism").
 *
 * One streaming pass over K worker (micro-batch) gradient buffers of a flat
 * parameter vector of length d produces the averaged gradient, its squared norm,
 * the between-worker variance sum, the paper's test statistic and next batch size,
 * and (fused variant) the AdamW update that consumes the averaged gradient.
 *
 * Notation: the paper writes J for the number of workers; this API writes K.
 *
 * Conventions that hold for every launching entry point
 *   - "device" pointers are memory of the CUDA device that is current on the calling
 *     thread ("grads" buffers, which are only read, may also be memory of a peer device that
 *     the current one can address); "host" pointers are ordinary memory read during the
 *     call only.
 *   - The caller owns every buffer.  The library allocates no device memory and
 *     keeps no state between calls that a result depends on (what it does keep, on the
 *     host: abs_last_cuda_error, and which kernel attributes it has set on which device).
 *   - Work is enqueued on `stream` (a cudaStream_t; NULL = the legacy default
 *     stream).  No call synchronises with the host; results are valid in stream order.
 *   - Return value: ABS_OK, or a negative abs_status.  Every status other than
 *     ABS_ERR_CUDA comes from a check made before anything is launched: no output was
 *     written.  ABS_ERR_CUDA reports a CUDA runtime call that failed.  A call enqueues one to
 *     three kernels; if the failing call was a launch after the first, the earlier kernels
 *     of the call may still run: the fused calls may then have updated params, m and v (and
 *     gbar_out) in place while stats_out and b_next_out were not written, and repeating the
 *     call would apply the update twice.  The refusal that can be foreseen is ruled out:
 *     whether the device can co-schedule the thread-block cluster of the final reduction is
 *     asked once per device before the first launch, and a single block is used if not.
 *     What remains is a launch refused because the context is already broken.
 *   - Aliasing: params, m and v are updated in place.  Apart from that, no output range may
 *     share a byte with a gradient buffer or with another output of the same call; the
 *     norm-test calls check this on the host and return ABS_ERR_ALIAS.
 *   - Results are deterministic: the same inputs give bit-identical outputs on every
 *     call, independent of how the hardware schedules thread blocks.
 */
#ifndef ABS_NORMTEST_H_
#define ABS_NORMTEST_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef void* abs_stream_t; /* a cudaStream_t */

typedef enum { ABS_F32 = 0, ABS_BF16 = 1 } abs_dtype;

typedef enum {
  ABS_OK = 0,
  ABS_ERR_NULL = -1,   /* a required pointer is NULL                                   */
  ABS_ERR_RANGE = -2,  /* K, d, b, ld, step, eta, b_cur or a hyper-parameter is out of range */
  ABS_ERR_SHARDS = -3, /* shard_offsets not non-decreasing, or ends are not 0 and d    */
  ABS_ERR_ALIGN = -4,  /* a buffer is not aligned to its element size                  */
  ABS_ERR_DTYPE = -5,  /* dtype is not an abs_dtype                                    */
  ABS_ERR_CUDA = -6,   /* a CUDA call failed; see abs_last_cuda_error()                */
  ABS_ERR_TOO_LARGE = -7, /* the problem needs more built-in scratch than the library holds */
  ABS_ERR_ALIAS = -8   /* an output overlaps a gradient buffer or another output        */
} abs_status;

enum { ABS_MAX_WORKERS = 1024, ABS_MAX_SHARDS = 128 };

/* AdamW hyper-parameters (alpha, beta1, beta2, epsilon, lambda of Algorithm 1). */
typedef struct {
  float lr;
  float beta1;
  float beta2;
  float eps;
  float weight_decay;
} abs_adamw_hparams;

/*
 * Layout of stats_out (device memory, doubles).  Header of ABS_STATS_HEADER doubles:
 */
enum {
  ABS_STAT_N2 = 0,      /* ||gbar||^2, gbar as written/consumed in fp32                  */
  ABS_STAT_S = 1,       /* sum_k ||g_k - gbar||^2   (per-sample form: sum over rows)     */
  ABS_STAT_Q = 2,       /* sum_k ||g_k||^2 (diagnostic: S = Q - K*n2); NaN = not computed */
  ABS_STAT_T = 3,       /* the statistic T                                               */
  ABS_STAT_FLAGS = 4,   /* ABS_FLAG_* bits stored as a double                            */
  ABS_STAT_NORM = 5,    /* K (worker form) or b-1 (per-sample form)                      */
  ABS_STAT_NCHUNKS = 6, /* number of reduction chunks the call used                      */
  ABS_STAT_ARGMAX = 7,  /* coordinate-wise calls: the coordinate with the largest T_i; else 0 */
  ABS_STATS_HEADER = 8
};
/* then n_shards records of ABS_SHARD_STRIDE doubles {n2_s, S_s, Q_s, 0}, in shard order,
 * then opaque scratch.  abs_stats_bytes() gives the total size.                        */
enum { ABS_SHARD_STRIDE = 4 };

enum {
  ABS_FLAG_DEGENERATE = 1, /* ||gbar||^2 == 0                                           */
  ABS_FLAG_NONFINITE = 2,  /* a sum is NaN or infinite; b_next = b_cur                  */
  ABS_FLAG_VIOLATED = 4    /* T > b_cur: the test failed and b_next = ceil(T)           */
};

/* Bytes the caller must provide for stats_out of abs_norm_test / abs_normtest_adamw:
 * header + shard records + chunk scratch.  Returns 0 on invalid arguments.  Host, pure. */
size_t abs_stats_bytes(int64_t d, int n_shards);

/* Bytes the caller must provide for stats_out of abs_persample_norm_test (b rows of d
 * columns): header + one shard record + the row-block work space + its ticket counters.
 * Returns 0 on invalid arguments.  Host, pure.                                          */
size_t abs_persample_stats_bytes(int64_t b, int64_t d);

/*
 * DDP-Norm / FSDP-Norm test (Sec. 3.2-3.3; Algorithm 1 from "Compute the batch
 * gradient" through the If/Else on T_k).
 *   gbar[i] = (1/K) sum_k g_k[i]                      (mean over workers, fp32 out)
 *   n2 = sum_i gbar[i]^2,  S = sum_k sum_i (g_k[i]-gbar[i])^2
 *   T = (S/K) / (eta^2 n2);   b_next = ceil(T) if T > b_cur else b_cur
 * The same sums are also reported per shard of the flat vector (FSDP-Norm: each
 * worker holds one parameter shard; Appendix A concatenates them); the totals are
 * the shard records added in shard order.
 *
 *   grads          host array of K device pointers, each d elements of `dtype`,
 *                  aligned to the element size (16-byte alignment is faster, not required).
 *                  They are only read, with plain loads and non-multicast bulk copies, so a
 *                  buffer may also live on another GPU whose memory the current device can
 *                  address (peer access enabled, or an opened inter-process handle): the
 *                  gradient exchange of Sec. 3.2 is then the kernel's own loads.  Every
 *                  output must be memory of the current device.
 *   K              1..ABS_MAX_WORKERS (1024 = 4 workers x 256 accumulation steps, the largest
 *                  layout of the paper's Table 5, should the J*M micro-batch gradients of a
 *                  step serve as the samples of the estimator)
 *   d              >= 1
 *   shard_offsets  host array of n_shards+1 non-decreasing offsets, [0]=0, [n_shards]=d;
 *                  NULL = one shard (n_shards ignored)
 *   n_shards       1..ABS_MAX_SHARDS
 *   eta            finite, > 0 (the paper uses 0.05-0.275; values >= 1 are accepted)
 *   b_cur          >= 1, the current global batch size
 *   stats_out      device, abs_stats_bytes(d, n_shards) bytes, 16-byte aligned
 *   gbar_out       device, d floats; must not overlap any grads[k] (ABS_ERR_ALIAS)
 *   b_next_out     device, one int64
 * Non-finite inputs are not an error: the flag is raised and b_next = b_cur.
 * The diagnostic Q is not computed (its slots read NaN): no decision uses it and it costs the
 * test, which is bound by instruction issue, 1-6% of its bandwidth.
 */
int abs_norm_test(const void* const* grads, int K, int64_t d, abs_dtype dtype,
                  const int64_t* shard_offsets, int n_shards, double eta, int64_t b_cur,
                  void* stats_out, float* gbar_out, int64_t* b_next_out, abs_stream_t stream);

/*
 * The norm test over gradients that arrive a few at a time (gradient accumulation: Sec. 3.2
 * names it for minibatches that exceed a worker's memory; Algorithm 1's accumulation loop), in
 * O(d) memory: the K new buffers are merged into the running mean of the count_in gradients
 * that the earlier calls of this step merged, and into the running variance sum.
 *
 *   count_in = 0     starts a step: `mean_inout` and the sums in `stats_inout` are only written.
 *   count_in > 0     `mean_inout` holds the mean of the count_in gradients so far and
 *                    `stats_inout` is the buffer the previous call of the step wrote (its shard
 *                    records carry the sums; the same d and shard table must be passed).
 * After the call `mean_inout` is the mean of all count_in + K gradients (after the last call of
 * the step: gbar of Algorithm 1), and the header, the shard records and b_next_out are those of
 * the test over all of them, with 1/(count_in + K) in place of 1/J in Eq. 5 -- what
 * abs_norm_test returns when given all the buffers at once, up to rounding: the running mean is
 * rounded to fp32 once per call (relative 2^-24 each, so gbar agrees with the one-call result
 * to about 2^-24 sqrt(calls) of its magnitude), the sums agree to the usual 1e-6.  Per call
 * K*s + 8 bytes per coordinate cross HBM (the new gradients once, the mean read and written).
 * The caller advances count_in by K between calls.  K is 1..64 here; Q is not computed.
 *
 *   mean_inout     device, d floats, aligned to 4 bytes; must not overlap a gradient buffer
 *   stats_inout    device, abs_stats_bytes(d, n_shards) bytes, 16-byte aligned
 *   other arguments as for abs_norm_test
 * Non-finite values, once merged, stay in the mean and the sums until a call with count_in = 0.
 */
int abs_norm_test_accumulate(const void* const* grads, int K, int64_t d, abs_dtype dtype,
                             const int64_t* shard_offsets, int n_shards, int64_t count_in,
                             double eta, int64_t b_cur, void* stats_inout, float* mean_inout,
                             int64_t* b_next_out, abs_stream_t stream);

/*
 * The closing call of a step in the carry-in form, fused with AdamW (Algorithm 1: the test,
 * then the AdamW lines on the batch gradient): merges the last K buffers as
 * abs_norm_test_accumulate does and applies the update with the final mean in the same pass,
 * so the mean is consumed in registers: K*s + 4 + 24 bytes per coordinate instead of
 * K*s + 8 for the merge plus 28 for abs_adamw_step.
 *
 *   mean_in        device, d floats: the running mean of the count_in gradients merged so far
 *                  (read only; NULL allowed when count_in = 0, which makes this call the whole
 *                  step, as abs_normtest_adamw is)
 *   gbar_out       device, d floats, or NULL when the final mean is not wanted; may be
 *                  `mean_in` itself (updated in place), must not overlap it otherwise
 *   params, m, v, hparams, step   as for abs_normtest_adamw
 * ABS_ERR_CUDA after the first launch: as for abs_normtest_adamw (the update may be enqueued).
 */
int abs_norm_test_accumulate_adamw(const void* const* grads, int K, int64_t d, abs_dtype dtype,
                                   const int64_t* shard_offsets, int n_shards, int64_t count_in,
                                   double eta, int64_t b_cur, void* stats_inout,
                                   const float* mean_in, float* gbar_out, int64_t* b_next_out,
                                   float* params, float* m, float* v,
                                   const abs_adamw_hparams* hparams, int64_t step,
                                   abs_stream_t stream);

/* abs_norm_test that also accumulates the diagnostic Q = sum_k sum_i g_k[i]^2, per shard and
 * in total (the identity S = Q - K*n2 checks a run's sums against each other). */
int abs_norm_test_q(const void* const* grads, int K, int64_t d, abs_dtype dtype,
                    const int64_t* shard_offsets, int n_shards, double eta, int64_t b_cur,
                    void* stats_out, float* gbar_out, int64_t* b_next_out, abs_stream_t stream);

/*
 * AdamW update (Algorithm 1, the five lines after the If/Else), in place, fp32:
 *   m = beta1 m + (1-beta1) g;  v = beta2 v + (1-beta2) g^2
 *   w = (1 - lr*wd) w - lr (m/(1-beta1^step)) / (sqrt(v/(1-beta2^step)) + eps)
 *   params, m, v   device, d floats each, updated in place
 *   gbar           device, d floats (e.g. gbar_out of abs_norm_test)
 *   hparams        host; lr, eps, weight_decay finite and >= 0; beta1, beta2 in [0,1)
 *   step           >= 1 (the k of Algorithm 1)
 */
int abs_adamw_step(float* params, const float* gbar, float* m, float* v, int64_t d,
                   const abs_adamw_hparams* hparams, int64_t step, abs_stream_t stream);

/*
 * AdamW on the gradient clipped by global norm -- what the paper's experiments add to
 * Algorithm 1 (Sec. 5 "gradient clipping"; "Gradient clipping 1.0" in the hyper-parameter
 * tables of Appendix C).  The paper prints no formula; this follows the convention of the
 * PyTorch routine its training stack calls:
 *   scale = min(1, max_norm / (||gbar|| + 1e-6));   then abs_adamw_step with scale*gbar.
 * ||gbar||^2 is read on the device from `stats_in`, the stats_out buffer that a preceding
 * abs_norm_test on the same stream wrote for this gbar (its ABS_STAT_N2 slot), so the
 * sequence norm test -> clipped update needs no host round trip.  Clipping needs the
 * global norm before the first coordinate is updated, which is why it is a second pass
 * (28 B per coordinate) and not part of the fused call.
 *   max_norm   finite, > 0;   stats_in  device, 8-byte aligned;   rest as abs_adamw_step
 */
int abs_adamw_step_clipped(float* params, const float* gbar, float* m, float* v, int64_t d,
                           const abs_adamw_hparams* hparams, int64_t step, double max_norm,
                           const void* stats_in, abs_stream_t stream);

/*
 * The fused step with the gradient clipped by the PREVIOUS step's global norm -- a single-pass
 * approximation of abs_norm_test + abs_adamw_step_clipped (40 instead of 48 B per coordinate at
 * K = 8 bf16).  It is NOT what the paper's experiments compute: they clip by the norm of the
 * gradient being applied, which is only known once the whole vector has been read; here
 *   scale = min(1, max_norm / (sqrt(n2_prev) + 1e-6)),  AdamW on scale * gbar,
 * with n2_prev = ||gbar||^2 of the step before, read on the device from `stats_prev` -- the
 * stats_out of the previous call.  stats_prev may be the very buffer passed as stats_out (its
 * header is read before this call's last kernel rewrites it); NULL = no clipping (the first
 * step).  The test's statistics and gbar_out are those of the unclipped gradient.  All other
 * arguments as abs_normtest_adamw; max_norm finite and > 0 when stats_prev is given.
 */
int abs_normtest_adamw_clip_prev(const void* const* grads, int K, int64_t d, abs_dtype dtype,
                                 const int64_t* shard_offsets, int n_shards, double eta,
                                 int64_t b_cur, void* stats_out, float* gbar_out,
                                 int64_t* b_next_out, float* params, float* m, float* v,
                                 const abs_adamw_hparams* hparams, int64_t step, double max_norm,
                                 const void* stats_prev, abs_stream_t stream);

/*
 * The fused step: abs_norm_test and abs_adamw_step in one pass, so gradients and
 * optimizer state cross HBM once.  Arguments as above; gbar_out may be NULL (the mean
 * then lives only in registers).  The diagnostic Q is not computed here: its slots in
 * stats_out read NaN.  Legal because the update uses only the mean gradient
 * and none of the test's results (Algorithm 1 lists the test first, with no data
 * dependence between the two).
 */
int abs_normtest_adamw(const void* const* grads, int K, int64_t d, abs_dtype dtype,
                       const int64_t* shard_offsets, int n_shards, double eta, int64_t b_cur,
                       void* stats_out, float* gbar_out, int64_t* b_next_out, float* params,
                       float* m, float* v, const abs_adamw_hparams* hparams, int64_t step,
                       abs_stream_t stream);

/*
 * The coordinate-wise norm test (Sec. 4: the test Proposition 1 and Theorem 1 are stated for;
 * Appendix B, first remark, prints it for the exact variance: for every coordinate i,
 * E[(d_i L_B - d_i L)^2] <= eta^2 (d_i L)^2).  The paper prints no sample form and runs the
 * summed test in its experiments; this is the sample form obtained the way Eq. 5 is obtained
 * from the exact-variance test -- coordinate i of the variance estimator displayed before
 * Eq. 5, divided by b, against eta^2 gbar_i^2:
 *   T_i = ((1/K) sum_k (g_k[i]-gbar[i])^2) / (eta^2 gbar[i]^2),  T = max_i T_i,
 *   b_next = ceil(T) if T > b_cur else b_cur
 * (the smallest batch size under which every coordinate would pass).  A coordinate with zero
 * variance has T_i = 0, also when gbar[i] = 0; positive variance with gbar[i] = 0 gives +inf.
 * T is never below the summed statistic of the same data (a weighted mean of the T_i).
 *
 * Same arguments as abs_norm_test / abs_normtest_adamw, same gbar, n2, S and (fused) AdamW
 * update, same traffic: the ratio is formed where the deviations and the mean already are.
 * What differs in stats_out: the Q slots read NaN; ABS_STAT_T is max_i T_i and
 * ABS_STAT_ARGMAX the lowest coordinate that attains it; ABS_STAT_FLAGS: NONFINITE (T = NaN,
 * b kept) when n2 or S is not finite, else DEGENERATE when n2 = 0 or T = +inf, VIOLATED when
 * T > b_cur; shard record s is {n2_s, S_s, argmax within the shard, max T_i within the shard}.
 * Accuracy: each ratio is formed in fp32 (hardware reciprocal), so T carries a relative error
 * of a few 1e-7 for up to 16 workers and up to about 1e-5 beyond (shifted one-pass
 * deviations); among coordinates whose ratios agree to that accuracy any one may be reported.
 * Ratios beyond the fp32 range (|gbar[i]| below about 1e-19 times the deviations) are
 * reported as +inf.
 */
int abs_norm_test_coordwise(const void* const* grads, int K, int64_t d, abs_dtype dtype,
                            const int64_t* shard_offsets, int n_shards, double eta, int64_t b_cur,
                            void* stats_out, float* gbar_out, int64_t* b_next_out,
                            abs_stream_t stream);
int abs_normtest_adamw_coordwise(const void* const* grads, int K, int64_t d, abs_dtype dtype,
                                 const int64_t* shard_offsets, int n_shards, double eta,
                                 int64_t b_cur, void* stats_out, float* gbar_out,
                                 int64_t* b_next_out, float* params, float* m, float* v,
                                 const abs_adamw_hparams* hparams, int64_t step,
                                 abs_stream_t stream);

/*
 * abs_normtest_adamw for callers that cannot allocate device memory.
 * (The paper has no counterpart: this is a deployment convenience, not part of the method.)
 *
 * Who needs it.  abs_normtest_adamw keeps its per-chunk partial sums in the tail of
 * stats_out, whose size grows with d, so the caller has to size and allocate that buffer
 * for every new problem size.  Some callers cannot: code that runs inside a region where
 * cudaMalloc is forbidden or would stall everything (a plugin's execute hook, a callback
 * on a latency-critical serving path, a process whose device memory is entirely owned by
 * another allocator), or a host that only has a fixed, small status buffer to offer.
 * This variant needs nothing that grows with d: the partial sums go to an array that is
 * part of the library image (ABS_NOALLOC_MAX_CHUNKS records of 32 bytes = 4 MiB, resident
 * on every GPU that loads the library until the process exits).  The call itself performs
 * no cudaMalloc/cudaFree and calls no allocating routine.
 *
 * Arguments, results and status codes are those of abs_normtest_adamw, except:
 *   stats_out   device, only (ABS_STATS_HEADER + n_shards*ABS_SHARD_STRIDE) doubles
 *               (header and shard records; no scratch tail), 16-byte aligned
 *   limit       the call's chunk count -- the sum over shards of ceil(shard length / c),
 *               c = 8192 for d >= 2^23 and 4096 below -- must not exceed
 *               ABS_NOALLOC_MAX_CHUNKS (any d up to about 1.07e9); larger problems return
 *               ABS_ERR_TOO_LARGE and launch nothing.  abs_noalloc_fits() answers the same
 *               question on the host without touching the GPU.
 * Both entry points run the same kernels on the same chunk layout, so on the same inputs
 * every output (statistics, shard records, b_next, gbar, params, m, v) is bit-identical to
 * abs_normtest_adamw's.
 *
 * Shared state.  All calls on one device use the same built-in array.  Nothing in it has
 * to be cleared between calls: every record the final reduction reads is written earlier
 * in the same call, so stale contents of a previous call are never observed.  But two
 * calls whose GPU work overlaps on one device (different streams, or several host threads)
 * race on it and produce undefined statistics: keep them on one stream or otherwise
 * ordered.
 * First call.  The first call on each device looks up the device address of the built-in
 * array (cudaGetSymbolAddress, with that device current; this may also trigger the lazy
 * load of the library's device code).  Make that first call outside of any stream
 * capture; later calls on the same device only launch kernels.  The address is cached for
 * the life of the process: it does not survive cudaDeviceReset() or the destruction of the
 * device's primary context, after which this entry point must not be used again.
 */
enum { ABS_NOALLOC_MAX_CHUNKS = 131072 };
/* 1 if abs_normtest_adamw_noalloc accepts this (d, shard table), 0 if it would return
 * ABS_ERR_TOO_LARGE or the arguments are invalid.  Host, pure. */
int abs_noalloc_fits(int64_t d, const int64_t* shard_offsets, int n_shards);
int abs_normtest_adamw_noalloc(const void* const* grads, int K, int64_t d, abs_dtype dtype,
                               const int64_t* shard_offsets, int n_shards, double eta,
                               int64_t b_cur, void* stats_out, float* gbar_out,
                               int64_t* b_next_out, float* params, float* m, float* v,
                               const abs_adamw_hparams* hparams, int64_t step,
                               abs_stream_t stream);

/*
 * Approximate norm test on per-sample gradients (Eq. 3, the Var definition before it,
 * and the b_{k+1} display after it) -- the single-device form of the test.
 *   G          device, row-major [b, ld] elements of `dtype`; row i = gradient of sample i;
 *              read once.  Rows that start on a 16-byte (fp32) / 8-byte (bf16) boundary take
 *              the fast path; any element-aligned matrix is accepted
 *   b          >= 2 rows (also the current batch size), d >= 1 columns, ld >= d
 *   dtype      ABS_F32 or ABS_BF16 (Sec. 5: the experiments train in bfloat16)
 *   gbar[c] = (1/b) sum_i G[i,c];  S = sum_i ||G[i,:]-gbar||^2;  ||Var||_1 = S/(b-1)
 *   T = ||Var||_1 / (eta^2 ||gbar||^2);  b_next = ceil(T) if T > b else b
 *   stats_out  device, abs_persample_stats_bytes(b, d) bytes, 16-byte aligned; header
 *              as above with NORM = b-1 and one shard record; the diagnostic Q is not
 *              computed (NaN).  The buffer must be ZERO-FILLED before its first use with
 *              this call: the thread blocks of its last kernel count themselves off in a
 *              ticket counter kept in this buffer (the doubles right after the shard record,
 *              at the same place for every b and d); the counter is back at zero when the call
 *              completes, so the buffer can be reused as it is, for any shape it is large
 *              enough for.  Zero it again after a call that returned ABS_ERR_CUDA.
 *   gbar_out   device, d floats;  b_next_out device, one int64
 */
int abs_persample_norm_test(const void* G, int64_t b, int64_t d, int64_t ld, abs_dtype dtype,
                            double eta, void* stats_out, float* gbar_out, int64_t* b_next_out,
                            abs_stream_t stream);

/*
 * The coordinate-wise test in its per-sample form (Sec. 4, Proposition 1: the condition is asked
 * of every coordinate, with the per-sample variance of that coordinate): the same pass over G,
 * the same gbar, n2 and S, but
 *   T_i = (sum_r (G[r,i]-gbar_i)^2 / (b-1)) / (eta^2 gbar_i^2),   T = max_i T_i
 * (T_i = 0 where the column has zero variance, +inf where only gbar_i = 0: then the test fails
 * for every batch size and b_next saturates, flag DEGENERATE).  The header's T slot holds T, its
 * ARGMAX slot the column where it occurs (the lowest one on a tie), the shard record is
 * {n2, S, that column, T}.  Arguments and the zero-filled stats buffer as for
 * abs_persample_norm_test.
 */
int abs_persample_norm_test_coordwise(const void* G, int64_t b, int64_t d, int64_t ld,
                                      abs_dtype dtype, double eta, void* stats_out,
                                      float* gbar_out, int64_t* b_next_out, abs_stream_t stream);

/*
 * The decision alone, on the host, from sums already reduced (e.g. to re-decide for a
 * different eta, or after combining per-rank sums in rank order).  Same expression
 * order as the device code: T = (S/norm) / ((eta*eta)*n2).  Writes T and the ABS_FLAG_*
 * bits when the pointers are non-NULL; returns b_next.  Pure.
 */
int64_t abs_decide(double S, double n2, double norm, double eta, int64_t b_cur, double* T_out,
                   int* flags_out);

/*
 * FSDP-Norm across processes (Sec. 3.3; Appendix A: the shard gradients are concatenated, so
 * the statistic is formed from the sums of all shards).  Each rank runs the norm test on its
 * own index range and contributes its three sums; every rank then calls this with the
 * gathered rows and obtains the same bits.
 *   per_rank    host, n_ranks rows of 3 doubles {n2_r, S_r, Q_r} in rank order
 *   totals_out  host, 3 doubles {n2, S, Q}: the rows added in rank order (the order in which
 *               the single-device call adds its shard records); may be NULL
 * Then the decision of abs_decide on the totals.  Returns b_next, or -1 when per_rank is NULL
 * or n_ranks < 1.  Pure.
 */
int64_t abs_combine_sums(const double* per_rank, int n_ranks, double norm, double eta,
                         int64_t b_cur, double* totals_out, double* T_out, int* flags_out);

/* Algorithm 1's rounding of a new batch size to the parallel layout:
 * micro = ceil(b/(J*M)), mini = M*micro, returns J*mini.  J, M >= 1.  Returns -1 on
 * invalid arguments.  Host, pure. */
int64_t abs_round_batch(int64_t b_next, int64_t J, int64_t M);

/*
 * Mixed precision (Sec. 5: the experiments train in bfloat16): the two update calls with one
 * more output, a bfloat16 copy of the updated parameters -- the working copy the next
 * forward pass reads while `params` stays the fp32 master -- written in the same pass
 * (+2 B per coordinate instead of a separate 6 B cast pass).  Each bf16 value is the fp32
 * value stored to `params`, rounded to nearest, ties to even.
 *   params_bf16_out  device, d 16-bit elements, 2-byte aligned (16-byte alignment keeps the
 *                    vector path); must not alias another argument
 * abs_normtest_adamw_mixed: all other arguments as abs_normtest_adamw.
 * abs_adamw_step_mixed: as abs_adamw_step; with stats_in non-NULL the gradient is clipped as
 * in abs_adamw_step_clipped (max_norm finite, > 0), with stats_in NULL max_norm is ignored.
 */
int abs_normtest_adamw_mixed(const void* const* grads, int K, int64_t d, abs_dtype dtype,
                             const int64_t* shard_offsets, int n_shards, double eta,
                             int64_t b_cur, void* stats_out, float* gbar_out, int64_t* b_next_out,
                             float* params, float* m, float* v, void* params_bf16_out,
                             const abs_adamw_hparams* hparams, int64_t step, abs_stream_t stream);
int abs_adamw_step_mixed(float* params, const float* gbar, float* m, float* v,
                         void* params_bf16_out, int64_t d, const abs_adamw_hparams* hparams,
                         int64_t step, double max_norm, const void* stats_in,
                         abs_stream_t stream);

/*
 * The batch-size schedule around the test (Algorithm 1: the While loop's counters and the
 * If branch; Sec. 5 "Training Specifications": a maximum global batch size above which the
 * test is no longer performed, and a test interval; Tables 5-7: base and maximum micro batch
 * size, base gradient accumulation steps).  Host-side integer state, no device work, no
 * allocation; the caller owns the struct and may read its fields.
 *
 *   J          workers (data-parallel size)
 *   M          gradient accumulation steps, grows when a new batch size needs a microbatch
 *              above max_micro
 *   micro      microbatch size b_{k,J}^M
 *   b          global batch size b_k = J*M*micro
 *   b_max      maximum global batch size
 *   max_micro  maximum micro batch size, 0 = no limit (M then never changes)
 *   interval   the test runs at steps k with k % interval == 0
 *   step       k, starts at 1;  samples = i, the samples processed so far
 *
 * abs_schedule_advance(s, b_test) closes step k: b_test is the b_next the test wrote (pass
 * s->b when no test ran).  With target = min(b_test, b_max):
 *   target <= b:  nothing changes (the Else branch);
 *   else          micro = ceil(target/(J*M));  if micro > max_micro > 0 then
 *                 M = ceil(target/(J*max_micro)), micro = ceil(target/(J*M));  b = J*M*micro
 *                 (the If branch); a b above b_max after rounding falls back to
 *                 micro = floor(b_max/(J*M)), and is dropped if that does not exceed the old b.
 * Then samples += the batch size step k used, step += 1.  The paper prints the rounding only;
 * the growth rule for M and the fallback at the cap are this library's reading.
 */
typedef struct abs_schedule {
  int64_t J, M, micro, b, b_max, max_micro, interval, step, samples;
} abs_schedule;

/* b = J*M*micro0 must not exceed b_max; micro0 must not exceed max_micro when that is set.
 * Returns ABS_OK, ABS_ERR_NULL or ABS_ERR_RANGE (also when b_max exceeds 2^60). */
int abs_schedule_init(abs_schedule* s, int64_t J, int64_t M, int64_t micro0, int64_t b_max,
                      int64_t max_micro, int64_t interval);
/* 1 if step s->step runs the test (b < b_max and step % interval == 0), else 0; -1 if s is NULL. */
int abs_schedule_test_due(const abs_schedule* s);
/* Returns ABS_OK, ABS_ERR_NULL, or ABS_ERR_RANGE (b_test < 1; the state is then unchanged). */
int abs_schedule_advance(abs_schedule* s, int64_t b_test);

/*
 * Self-test of the bounded waits (no counterpart in the paper).  The staged kernels wait for
 * their asynchronous copies on shared-memory barriers, and every such wait gives up after a
 * fixed number of polls (2^18, about one second on a B200) instead of spinning for ever; a kernel whose wait gave up
 * poisons its partial sums, so the call reports ABS_FLAG_NONFINITE.  This entry point runs
 * that wait on a barrier nothing will complete, for `polls` polls (1 .. 2^18), and writes
 * out[0] = 1 if the wait gave up (it must), out[1] = the time it took in nanoseconds
 * (device, two int64).  It shows that the give-up path ends by itself and how long the full
 * limit lasts on the device at hand.
 */
int abs_selftest_bounded_wait(int polls, int64_t* out, abs_stream_t stream);

const char* abs_status_string(int status);

/* The cudaError_t of the most recent ABS_ERR_CUDA on this thread (0 if none). */
int abs_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* ABS_NORMTEST_H_ */
