/*
 * abs.h -- C ABI of the adaptive-batch-size test and the fused local-optimiser
 * kernels for NVIDIA B200 (sm_100a).
 *
 * The library implements the per-round batch-size test of the adaptive local
 * batch size method for local gradient methods and the parameter updates around
 * it, for M simulated workers held as replicas on ONE GPU:
 *
 *   abs_test_stats     mean gradient, norm-test variance, inner-product and
 *                      orthogonality variances of per-sample gradients
 *                      (Eq. batch_grad, Eq. def_var, Eq. approx_norm_local)
 *   abs_next_batch     the ceilings T^m, max{T, b}, the maximum over workers and
 *                      the cap (Eq. norm_test, Eq. test_stat, Algorithm 1)
 *   local_sgd_step     x^m <- x^m - alpha g^m           (Eq. local_sgd_alt, line 1)
 *   local_adamw_step   AdamW inner optimiser             (Section 4.2, Appendix C.2)
 *   local_shb_step     momentum-SGD inner optimiser      (Section 6.1)
 *   replica_average    x^m <- (1/M) sum_m x^m            (Eq. local_sgd_alt, line 2)
 *
 * Conventions
 *   - Every function returns an int: ABS_OK (0) or a negative ABS_ERR_* code.
 *     Nothing throws across this boundary.  abs_last_error() gives a message.
 *   - Unless a parameter says "host", every tensor pointer is a DEVICE pointer
 *     owned by the caller, on the device the context was created for.
 *   - Calls only enqueue work on `stream` (a cudaStream_t passed as void*; NULL
 *     is the legacy default stream).  They do not synchronise; results are
 *     valid in stream order.  The *_host variants are the exception: they copy,
 *     run and synchronise before returning.
 *   - A context owns a workspace for per-CTA partial sums.  Calls that use the
 *     same context must be issued in stream order on one stream at a time.
 *   - Data-dependent conditions (non-finite input, zero mean gradient, a
 *     copy that never completed) are reported in abs_stats.status on the
 *     device; they never trap.
 *   - Strides are in ELEMENTS of the tensor's type.  All index arithmetic is
 *     64-bit.
 */
#ifndef ABS_H_
#define ABS_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- error codes ---------------------------------------------------------- */
#define ABS_OK                0
#define ABS_ERR_INVALID_ARG  -1   /* null pointer, b < 2, d < 1, stride < extent, ...        */
#define ABS_ERR_UNSUPPORTED  -2   /* shape outside what the kernels cover (stated per call)  */
#define ABS_ERR_WORKSPACE    -3   /* the context's workspace is too small for this call      */
#define ABS_ERR_CUDA         -4   /* a CUDA runtime / driver call failed                     */
#define ABS_ERR_NO_DEVICE    -5   /* no usable sm_100 device; there is no CPU fallback       */

/* ---- status bits written to abs_stats.status ------------------------------ */
#define ABS_STATUS_NONFINITE  1u  /* an input or an accumulator was not finite (or overflowed) */
#define ABS_STATUS_ZERO_MEAN  2u  /* ||gbar||^2 == 0: the test ratios are undefined            */
#define ABS_STATUS_NORM_ONLY  8u  /* a record merged from sub-batches: only gbar_sq, var_norm,
                                     sum_sq and rows are meaningful (abs_stats_merge)          */
#define ABS_STATUS_TIMEOUT    4u  /* an asynchronous tile copy did not arrive in time; the
                                     numbers in this record are not valid                      */

typedef struct abs_ctx abs_ctx;   /* opaque */

/* Creates a context bound to CUDA device `device` (must be compute capability
 * 10.x; otherwise ABS_ERR_NO_DEVICE).  workspace_bytes = 0 selects the default
 * (64 MiB), enough for b <= 4096 rows and M <= 64 workers.  The context owns
 * its device allocations until abs_destroy. */
int abs_create(abs_ctx** out, int device, size_t workspace_bytes);
int abs_destroy(abs_ctx* ctx);

/* Message of the last failing call on this context (host string, owned by the
 * context, valid until the next call).  ctx may be NULL: then the message of the
 * last failing abs_create on this thread. */
const char* abs_last_error(const abs_ctx* ctx);

/* Optional tuning of the statistics kernels; 0 restores the automatic
 * choice.  key: "stats_stages" (2..8 tile buffers), "stats_ctas_per_worker",
 * "stats_force_generic" (1 = always use the alignment-free kernel),
 * "stats_flush_every" (tiles between fp64 flushes of the per-row sums; for the
 * tcgen05 kernel: tiles added up in its fp32 accumulators before the fold into
 * fp64, at most 64),
 * "stats_stage_kb" (upper bound on one tile buffer, 4..200 KiB),
 * "stats_timeout_cycles" (SM clock cycles a wait for a tile copy may last before
 * the record is flagged ABS_STATUS_TIMEOUT; default about two seconds),
 * "stats_fault_drop_loads" (fault injection for tests: the loaders of the tiled,
 * cluster and tcgen05 kernels issue no copies, abs_logreg_rounds_fused sends no
 * partial gradients and the tensor-core products of the MLP producer fill no
 * operand tile, so every wait runs out and the records come back flagged
 * ABS_STATUS_TIMEOUT; nothing traps or hangs),
 * "stats_cluster_rows" (target rows per CTA of the cluster kernel, 16..512),
 * "stats_no_cluster" (1 = do not split the rows of a batch over a thread-block
 * cluster when b > 256),
 * "mlp_no_tensor_cores" (1 = the matrix products of the MLP producer run on the
 * CUDA cores in fp32 with fp64 folding instead of on the tensor cores),
 * "stats_no_secondary" (1 = the cluster kernel leaves the SMs idle that its
 * clusters cannot occupy instead of giving them a second launch of two-CTA
 * clusters), "stats_secondary_pct" (the speed of an SM of that second launch in
 * per cent of an SM of the first, which sets its share of the columns; 0 = 95, or 80 for rows
 * more than 64 MB apart),
 * "stats_no_gram" (1 = do not use the tensor-core Gram kernels for bf16, b <= 256),
 * "stats_no_recheck" (1 = keep a Gram kernel's record even when its sums are
 * ill-conditioned, i.e. never recompute it with the tiled kernel),
 * "stats_ctas_per_sm" (1: one CTA per SM, 64 KiB buffers, up to 16 rows per
 * thread; 2: two CTAs per SM, 32 KiB buffers, up to 8 rows per thread).
 * Unknown key or out-of-range value: ABS_ERR_INVALID_ARG. */
int abs_set_tuning(abs_ctx* ctx, const char* key, long long value);

typedef enum { ABS_F32 = 0, ABS_BF16 = 1 } abs_dtype;

/* One record per worker, written by abs_test_stats.  With rows g_1..g_b of one
 * worker, gbar = (1/b) sum_i g_i (Eq. batch_grad), N = ||gbar||^2,
 * c_i = <g_i, gbar>:                                                           */
typedef struct {
  double gbar_sq;     /* N                                                       */
  double var_norm;    /* 1/(b-1) sum_i ||g_i - gbar||^2          (Eq. def_var)   */
  double var_ip;      /* 1/(b-1) sum_i (c_i - mean_i c_i)^2      (Eq. def_var of c_i) */
  double var_orth;    /* 1/(b-1) sum_i ||o_i - mean o||^2, o_i = g_i - (c_i/N) gbar;
                         evaluated as var_norm - var_ip / N (equal by orthogonality);
                         equals var_norm when N == 0                              */
  double sum_sq;      /* sum_i ||g_i||^2 = (b-1) var_norm + b N                  */
  long long rows;     /* b                                                       */
  unsigned status;    /* ABS_STATUS_* bits                                       */
  unsigned recomputed;/* 1: the tensor-core Gram kernel's sums were too ill-conditioned
                         (rows dominated by a common vector) and the record comes
                         from a second, centred pass over G; else 0              */
} abs_stats;          /* 56 bytes */

/* Batch-size test statistics of M workers (Eq. def_var applied per worker,
 * Eq. approx_norm_local; Algorithm 1, variance step).
 *   G            [M][b][d] per-sample (or per-micro-batch) gradients, dtype fp32
 *                or bf16; element (m,i,j) at G[m*worker_stride + i*row_stride + j]
 *   M >= 1, b >= 2 (the variance divides by b-1), d >= 1,
 *   row_stride >= d, worker_stride >= (b-1)*row_stride + d (ignored if M == 1)
 *   gbar_out     optional [M][d] fp32 (contiguous, worker m at gbar_out + m*d):
 *                receives the batch gradients; may be NULL
 *   stats_out    [M] records
 * G is read exactly once from HBM when its base address and both strides are
 * multiples of 16 bytes and b <= 4096 (bf16 input with b <= 256 goes through
 * tensor-core Gram-matrix kernels, other input with b > 256 through a kernel
 * that splits the rows over a thread-block cluster, everything else through the
 * tiled kernel); otherwise an alignment-free kernel that reads it twice is used.
 * The result does not depend on which kernel ran beyond floating-point rounding.
 * Accumulation: fp32 within a tile (the Gram kernels: exact bf16 products added
 * in fp32 over at most 8192 columns), fp64 across tiles; the reduction order is
 * fixed, so repeated calls give bit-identical records.
 * The Gram kernels only see uncentred products, so their variance is a difference
 * of two sums of size sum_i ||g_i||^2: when b N exceeds a few tens (tcgen05) or a
 * few thousand (mma.sync) times (b-1) var_norm -- rows dominated by a common
 * vector -- or N exceeds about 2e5 sqrt(var_ip), the finalisation flags the
 * result on the device and the tiled kernel, which accumulates centred values,
 * recomputes it in a second pass (abs_stats.recomputed = 1).  The two guarded
 * launches are always enqueued and return at once when not needed, so the call
 * stays free of host synchronisation.
 * Errors: ABS_ERR_INVALID_ARG, ABS_ERR_WORKSPACE, ABS_ERR_CUDA.               */
int abs_test_stats(abs_ctx* ctx, const void* G, abs_dtype dtype, int M, long long b, long long d,
                   long long row_stride, long long worker_stride,
                   float* gbar_out, abs_stats* stats_out, void* stream);

/* What abs_test_stats would launch for a shape: the host-side planning of the
 * statistics kernels, exposed for inspection and for tests that need no GPU.
 * aligned != 0 means base address and strides are multiples of 16 bytes.          */
typedef struct {
  int route;              /* 0 Gram (bf16, 7 <= b <= 32), 1 cluster, 2 tiled, 3 generic two-sweep,
                             4 Gram on tcgen05 (bf16, 32 < b <= 256)                          */
  int lanes_per_row;      /* 16-byte vectors per tile row: a tile row has 16*lanes_per_row bytes */
  int warps_per_box;      /* consumer warps that share one box of rows                        */
  int boxes_per_stage;
  int stages;             /* tile buffers in the ring                                         */
  int box_rows;           /* rows of one TMA box (<= 256)                                     */
  int row_boxes;          /* boxes stacked to cover the rows of a tile                        */
  int rows_per_thread;
  int keep_in_registers;  /* the tile stays in registers between the two sweeps               */
  int full;               /* every thread owns exactly rows_per_thread rows                   */
  int cluster_size;       /* CTAs per cluster (1 outside the cluster route)                   */
  int rows_per_cta;
  unsigned stage_bytes;
  unsigned reserved;
  size_t smem_bytes;      /* dynamic shared memory per CTA                                    */
} abs_stats_plan;
int abs_plan_stats(abs_dtype dtype, long long b, int aligned, int sm_count, size_t smem_optin,
                   abs_stats_plan* out);

/* Same computation for HOST buffers: G_host is copied to a device buffer owned
 * by the context (grown on demand), the statistics are computed and copied back
 * to stats_host [M] and, if not NULL, gbar_host [M][d]; the call returns after
 * everything has completed.  G_host is contiguous ([M][b][d], row_stride = d).
 * Pinned host memory makes the copies faster but is not required.
 * stats_dev / gbar_dev are optional DEVICE buffers ([M] records, [M][d] fp32) that
 * receive the same results on the device, for a following abs_next_batch /
 * local_*_step that should not wait for another host-to-device copy.            */
int abs_test_stats_host(abs_ctx* ctx, const void* G_host, abs_dtype dtype, int M, long long b,
                        long long d, float* gbar_host, abs_stats* stats_host,
                        float* gbar_dev, abs_stats* stats_dev, void* stream);

/* Statistics without any allocation.  (The paper has no counterpart: this entry
 * point exists for the sake of the calling program, not of the method.)
 *
 * abs_create allocates a device workspace, and cudaMalloc / cudaFree synchronise the
 * device.  Some callers cannot accept that: programs whose device memory is handed
 * out entirely by their own pool, plug-ins that run under a fixed memory budget,
 * latency-critical sections that must not hit an implicit device synchronisation.
 * For them this call computes the same statistics as abs_test_stats (the same
 * records up to floating-point rounding: it only uses the tiled kernel and the
 * alignment-free kernel, so bf16 input with b <= 256 and any input with b > 256
 * take another, slower kernel than in the context call), takes no
 * context, and keeps its scratch (per-CTA partial sums and a status word) in a
 * fixed array of ABS_NOALLOC_SCRATCH_BYTES + 256 bytes that is part of the library
 * image: every GPU on which the library is loaded holds that array until the
 * process exits, used or not.
 *   - Arguments and results as for abs_test_stats; the device used is the CURRENT
 *     CUDA device of the calling thread, and all pointers must belong to it.
 *   - Limits: b <= ABS_NOALLOC_MAX_ROWS and M <= ABS_NOALLOC_MAX_WORKERS; larger
 *     problems are refused with ABS_ERR_UNSUPPORTED (message from
 *     abs_noalloc_last_error) and need abs_test_stats with a context.
 *   - The first call on each device looks up the device address of the array and a
 *     few device attributes (no allocation by this library; a CUDA runtime that
 *     loads modules lazily places the array on the GPU at this moment).  Make that
 *     first call during start-up, outside any stream capture.
 *   - All calls on one device share the one array.  It still holds the previous
 *     call's partial sums; the call clears what has to start at zero itself.  Two
 *     calls that can run on the GPU at the same time (different streams, different
 *     host threads) would overwrite each other's partial sums: issue them in one
 *     stream, or order them with events.
 *   - Calls no cudaMalloc, cudaFree or other allocating routine.                    */
#define ABS_NOALLOC_SCRATCH_BYTES (8u << 20)
#define ABS_NOALLOC_MAX_ROWS      2048
#define ABS_NOALLOC_MAX_WORKERS   64
int abs_test_stats_noalloc(const void* G, abs_dtype dtype, int M, long long b, long long d,
                           long long row_stride, long long worker_stride,
                           float* gbar_out, abs_stats* stats_out, void* stream);
/* Message of the last failing abs_test_stats_noalloc call on this thread. */
const char* abs_noalloc_last_error(void);

typedef enum {
  ABS_TEST_NORM = 0,               /* norm test on the rows of G (Eq. approx_norm_local)               */
  ABS_TEST_AUG_INNER_PRODUCT = 1,  /* augmented inner-product test on the rows of G                    */
  ABS_TEST_NORM_WORKERS = 2        /* Algorithm 2 ("actual implementation"): the norm test on the M
                                      workers' BATCH gradients (Eq. test_stat_actual).  For
                                      abs_next_batch it is the norm test (the caller sets row_weight =
                                      local batch size and divisor = M); the per-round drivers
                                      abs_logreg_round / abs_mlp_round form the statistics themselves
                                      from the batch gradients of the round's last local step          */
} abs_test_kind;

typedef struct {
  int kind;             /* abs_test_kind                                              */
  int reserved;         /* zero                                                       */
  double eta;           /* norm test constant (Eq. approx_norm)                       */
  double theta;         /* inner-product test constant                                */
  double nu;            /* orthogonality test constant                                */
  long long b_max;      /* maximum local batch size (cap), >= 1                       */
  double row_weight;    /* samples one row stands for: 1 for per-sample gradients, the
                           micro-batch size for micro-batch gradients, the local batch
                           size when rows are workers' batch gradients (Section 4.3)   */
  double divisor;       /* 1, or M for Eq. test_stat_actual / Algorithm 2              */
} abs_test_cfg;

/* Next local batch size (Eq. norm_test, Eq. test_stat, Algorithm 1: b <- max{T, b};
 * display below Eq. test_stat: maximum over workers).  Per worker m, in fp64,
 *   norm test        T^m = ceil( s/D * var_norm / (eta^2 N) )
 *   augmented ip     T^m = max( ceil( s/D * var_ip / (theta^2 N^2) ),
 *                               ceil( s/D * var_orth / (nu^2 N) ) )
 * with s = row_weight, D = divisor; 0/x counts as 0 (also 0/0), x/0 as +infinity;
 * ceilings saturate at 2^62; a record flagged NONFINITE or TIMEOUT gives T^m = 0.
 *   b_next = min( b_max, max( b_cur, max_m T^m ) ).
 *   stats   [M] device records;  cfg  HOST pointer (copied by value at the call)
 *   b_cur   device, 1 value;  T_out device [M] or NULL;  b_next device, 1 value
 *           (may alias b_cur).  M <= 1024.                                          */
int abs_next_batch(abs_ctx* ctx, const abs_stats* stats, int M, const abs_test_cfg* cfg,
                   const long long* b_cur, long long* T_out, long long* b_next, void* stream);

/* Per-worker next local batch sizes (Eq. test_stat before the practical maximum
 * over workers; Algorithm 1: b^m <- max{T^m, b^m}), with one norm-test constant
 * per worker (eta_m of Eq. approx_norm_local):
 *   b_next[m] = min( b_max, max( b_cur[m], T^m ) ),  T^m as in abs_next_batch.
 * eta_m: DEVICE array [M] of constants, or NULL to use cfg->eta for every worker
 * (ignored by the augmented inner-product test).  b_cur, b_next, T_out: device [M]
 * (b_next may alias b_cur; T_out may be NULL).  cfg is a HOST pointer.            */
int abs_next_batch_local(abs_ctx* ctx, const abs_stats* stats, int M, const abs_test_cfg* cfg,
                         const double* eta_m, const long long* b_cur, long long* T_out,
                         long long* b_next, void* stream);

/* Norm-test statistics of a batch that arrives in sub-batches (gradient
 * accumulation over micro-batches, Section 6): folds sub-batch b into the running
 * pair a.  Per worker m, with n = rows, S = (n-1) var_norm (Eq. def_var):
 *   mean_a <- (n_a mean_a + n_b mean_b) / (n_a + n_b)                  (in place)
 *   S      <- S_a + S_b + ||mean_a - mean_b||^2 n_a n_b / (n_a + n_b)
 * rec_a [M] receives rows, var_norm, gbar_sq = ||mean||^2, sum_sq and the status
 * bit ABS_STATUS_NORM_ONLY (var_ip / var_orth cannot be merged: they are set to 0
 * and abs_next_batch gives T = 0 for the augmented test on such a record).
 * mean_a, mean_b: [M][d] fp32 batch gradients as written by abs_test_stats
 * (gbar_out); rec_a, rec_b: the matching records.  All device pointers.           */
int abs_stats_merge(abs_ctx* ctx, float* mean_a, const float* mean_b, int M, long long d,
                    abs_stats* rec_a, const abs_stats* rec_b, void* stream);

/* Local SGD step for all replicas (Eq. local_sgd_alt): X[m] <- X[m] - lr * Gb[m],
 * m < M, in fp32.  X, Gb: [M][d] fp32 with replica m at + m*replica_stride
 * (>= d).  average_after != 0 fuses the model averaging of the round's last step:
 * every replica receives (1/M) sum_m (X[m] - lr*Gb[m]) at no extra memory traffic.
 * X is updated in place.                                                        */
int local_sgd_step(abs_ctx* ctx, float* X, const float* Gb, int M, long long d,
                   long long replica_stride, float lr, int average_after, void* stream);

typedef struct {
  float lr, beta1, beta2, eps, weight_decay;
  int reserved;       /* zero */
  long long step;     /* t >= 1, shared by all replicas, keeps counting across rounds */
} abs_adamw_cfg;

/* Local AdamW step for all replicas (inner optimiser of Section 4.2 / Appendix
 * C.2; rule of the cited optimiser, decoupled weight decay):
 *   m <- beta1 m + (1-beta1) g ;  v <- beta2 v + (1-beta2) g^2
 *   x <- x (1 - lr wd) - lr (m / (1-beta1^t)) / ( sqrt(v / (1-beta2^t)) + eps )
 * X, Mom1, Mom2, Gb: [M][d] fp32, same replica_stride; all but Gb updated in place.
 * average_after != 0: X[m] <- mean over replicas of the updated X; the moments
 * stay local.  cfg is a HOST pointer.                                           */
int local_adamw_step(abs_ctx* ctx, float* X, float* Mom1, float* Mom2, const float* Gb, int M,
                     long long d, long long replica_stride, const abs_adamw_cfg* cfg,
                     int average_after, void* stream);

/* Local stochastic-heavy-ball (momentum SGD) step, the inner optimiser of the
 * paper's image experiments (Section 6.1):
 *   g <- g + wd x ;  u <- momentum u + g ;  x <- x - lr u
 * X, Buf (the momentum buffer u), Gb: [M][d] fp32.                              */
int local_shb_step(abs_ctx* ctx, float* X, float* Buf, const float* Gb, int M, long long d,
                   long long replica_stride, float lr, float momentum, float weight_decay,
                   int average_after, void* stream);

/* Model averaging (Eq. local_sgd_alt, second line; Algorithm 1 "update the
 * global model"): every replica receives (1/M) sum_m X[m], in place.            */
int replica_average(abs_ctx* ctx, float* X, int M, long long d, long long replica_stride,
                    void* stream);

/* ---- the outer loop: sample counter, stop rule, cadence of the test ---------------------- */

/* The counters of Algorithm 1 / Algorithm 2, kept on the DEVICE so that rounds can follow one
 * another without a host read-back: B (samples processed), k (rounds completed) and the N of
 * "while B < N".  The caller allocates it in device memory, initialises it and may copy it back
 * at any time.  The drivers add, per round, sum_m sum_h b^m_{k,h} (Algorithm 1) -- which is
 * H M b_k when the size is shared and constant over a round (Algorithm 2) -- and 1 to k.
 * abs_logreg_rounds_fused_opts also obeys the stop rule on the device: it runs no round once
 * samples >= n_stop (n_stop <= 0: no stop).  The enqueue-only per-round drivers cannot skip
 * launches that are already enqueued; their caller reads the block back with the batch size. */
typedef struct {
  long long samples;    /* B                                                          */
  long long rounds;     /* k                                                          */
  long long n_stop;     /* N; <= 0: never stop                                        */
  long long reserved;   /* zero                                                       */
} abs_round_ctl;

/* Cadence and ownership of the batch size (HOST struct, copied at the call).         */
typedef struct {
  int test_every_step;  /* 0: the test once per round, on the last local step's gradients
                           (Section 4.3, last paragraph); 1: after every local step, the
                           next step already using the new size (Algorithm 1)          */
  int per_worker;       /* 1: b^m <- max{T^m, b^m} per worker (Eq. test_stat, Algorithm 1);
                           0: every worker continues with the maximum over the workers
                           (display below Eq. test_stat)                               */
  const double* eta_m;  /* DEVICE [M] norm-test constants eta_m (Eq. approx_norm_local), or
                           NULL: cfg->eta for every worker                             */
  abs_round_ctl* ctl;   /* DEVICE counter block, or NULL                               */
} abs_round_opts;

/* samples += times * (sizes[0] + ... + sizes[n-1]);  rounds += add_rounds  -- one tiny launch.
 * ctl, sizes: device.                                                                */
int abs_round_count(abs_ctx* ctx, abs_round_ctl* ctl, const long long* sizes, int n, long long times,
                    long long add_rounds, void* stream);

/* ---- producers and round drivers for the synthetic end-to-end problems ------------------ */

/* Per-sample gradients of the logistic loss (Algorithm 1, per-sample gradient
 * step): row i of worker m is (sigmoid(a^T x^m) - y) a with a = A[idx[m][i]].
 *   A [n][d] fp32 features, y [n] fp32 labels in {0,1}, idx [M][idx_stride] int32
 *   sample indices (the first b of each row are used), X [M][d] parameters,
 *   G [M][b][d] output (contiguous).                                              */
int abs_logreg_grads(abs_ctx* ctx, const float* A, const float* y, long long n, long long d,
                     const int* idx, long long idx_stride, const float* X, int M, long long b,
                     float* G, void* stream);

/* One communication round of local SGD on the logistic problem (Algorithm 2's
 * structure, Algorithm 1's per-sample statistic evaluated once per round, Section
 * 4.3): for h < H: per-sample gradients of batch idx[h] -> statistics and batch
 * gradient -> local SGD step (the last one fused with the model averaging); then
 * the batch-size update from the statistics of the last local step.
 *   idx [H][M][idx_stride] int32;  b the current batch size (host value, equal to
 *   *b_dev);  G_scratch [M][b][d], Gb_scratch [M][d], stats [M], T_out [M] or NULL;
 *   b_dev device int64: holds b on entry and the next batch size afterwards.
 *   ctl device counter block or NULL: B += H M b (Algorithm 2's counter), k += 1.
 * cfg->kind == ABS_TEST_NORM_WORKERS runs Algorithm 2 as printed: no per-sample test; after
 * the averaging the M batch gradients of the last local step (rows of Gb_scratch) give
 * Var = b/(M-1) sum_m ||g^m - gbar||^2 and T = ceil(Var / (M eta^2 ||gbar||^2)); needs M >= 2;
 * stats[0] receives that record (rows = M), T_out[0] the T, the other entries are unspecified.
 * Only enqueues; read b_dev (and ctl) back before sizing the next round.          */
int abs_logreg_round(abs_ctx* ctx, const float* A, const float* y, long long n, long long d,
                     const int* idx, long long idx_stride, float* X, int M, int H, long long b,
                     float lr, const abs_test_cfg* cfg, float* G_scratch, float* Gb_scratch,
                     abs_stats* stats, long long* T_out, long long* b_dev, abs_round_ctl* ctl,
                     void* stream);

/* The same round with the test after every local step (Algorithm 1 as printed): at step h
 * worker m draws b^m_{k,h} samples, its statistics give T^m_{k,h}, and step h + 1 runs with
 * b^m_{k,h+1} = min(b_max, max{T^m, b^m}) -- per worker, or the maximum over the workers
 * for all of them (opts->per_worker).  opts may be NULL (shared size, cfg->eta, no counter).
 *   b_host  HOST array [M]: the sizes the round starts with; on return the sizes after it
 *   b_dev   device [M] scratch that holds the same values
 *   idx [H][M][idx_stride] with idx_stride >= cfg->b_max;  G_scratch room for M * b_max rows
 *   of d floats;  stats [H][M] and T_out [H][M] (or NULL): the records and T of every step.
 * The grids of step h + 1 depend on sizes decided on the device in step h, so this call
 * WAITS for the stream once per local step to read M integers back (the one driver of the
 * library that synchronises; abs_logreg_rounds_fused_opts does the same work without).   */
int abs_logreg_round_per_step(abs_ctx* ctx, const float* A, const float* y, long long n, long long d,
                              const int* idx, long long idx_stride, float* X, int M, int H,
                              long long* b_host, float lr, const abs_test_cfg* cfg,
                              const abs_round_opts* opts, float* G_scratch, float* Gb_scratch,
                              abs_stats* stats, long long* T_out, long long* b_dev, void* stream);

/* `rounds` communication rounds of the same method in ONE cooperative launch
 * (Algorithm 2's structure, Algorithm 1's per-sample statistic once per round,
 * Section 4.3; b <- min(b_max, max{b, max_m T_m})): the parameters stay in shared
 * memory, the batch size stays on the device from round to round, the per-sample
 * gradient matrix is never written, and there is one grid-wide barrier per round
 * (none inside a local step).  For small problems, where abs_logreg_round is bound by launch latency.
 *   idx [rounds][H][M][idx_stride] int32 with idx_stride >= cfg->b_max (indices
 *   outside [0, n) are clamped);  X [M][d] in place (replica stride d);
 *   stats [rounds][M] records of each round's test;  T_out [rounds][M] or NULL;
 *   b_hist [rounds + 1] or NULL: the batch size each round ran with, then the last
 *   update;  b_dev: the starting size on entry (raised to 2, capped at b_max), the
 *   size after the last round on exit.
 * Needs d <= 1024, d % 4 == 0, M <= 64 and 16-byte aligned A and X, else
 * ABS_ERR_UNSUPPORTED; scratch comes from the context's workspace
 * (ABS_ERR_WORKSPACE if it is too small).  Each worker is one thread-block cluster
 * and the launch is cooperative (all CTAs resident); ABS_ERR_UNSUPPORTED if the
 * device cannot hold M clusters at once, ABS_ERR_CUDA if it refuses the launch.
 * The CTAs of a cluster wait for one another's partial gradients with the limit of
 * the "stats_timeout_cycles" tuning key; a wait that runs out never hangs the
 * launch: the records of that round and of the following ones carry
 * ABS_STATUS_TIMEOUT, which gives T = 0, and the parameters are then not to be
 * used.  Only enqueues.                                                            */
int abs_logreg_rounds_fused(abs_ctx* ctx, const float* A, const float* y, long long n, long long d,
                            const int* idx, long long idx_stride, int rounds, float* X, int M, int H,
                            float lr, const abs_test_cfg* cfg, abs_stats* stats, long long* T_out,
                            long long* b_hist, long long* b_dev, void* stream);

/* The same launch with the cadence, the ownership of the batch size, per-worker constants
 * and the counters of Algorithm 1 / Algorithm 2 chosen by `opts` (HOST pointer; NULL gives
 * abs_logreg_rounds_fused).  With opts:
 *   b_dev   device [M]: every worker's size on entry and after the last round that ran
 *   test once per round:   stats, T_out [rounds][M];  b_hist [rounds][M] (or NULL): the size
 *                          each round ran with
 *   test_every_step:       stats, T_out, b_hist [rounds][H][M]: record, T and the size of
 *                          every local step (Algorithm 1); one cluster-wide barrier per step
 *                          more, and a grid-wide one per step when the size is shared
 *   cfg->kind == ABS_TEST_NORM_WORKERS (with or without opts; not with test_every_step or
 *                          per_worker; M >= 2): Algorithm 2 as printed -- no per-sample
 *                          statistics, the norm test on the M batch gradients of the round's
 *                          last local step after the averaging; per round stats[.][0] holds that
 *                          record (rows = M, flagged ABS_STATUS_NORM_ONLY) and T_out[.][0] the T
 *   opts->ctl              B and k are read at the start and written back at the end; no
 *                          round starts once B >= n_stop (entries of rounds that did not
 *                          run are left untouched); X holds x_{K,0} of the last round run.  */
int abs_logreg_rounds_fused_opts(abs_ctx* ctx, const float* A, const float* y, long long n, long long d,
                                 const int* idx, long long idx_stride, int rounds, float* X, int M,
                                 int H, float lr, const abs_test_cfg* cfg, const abs_round_opts* opts,
                                 abs_stats* stats, long long* T_out, long long* b_hist,
                                 long long* b_dev, void* stream);

/* Three-layer ReLU MLP with softmax cross-entropy (the second synthetic problem).
 * dims = {n0, n1, n2, n3} layer widths.  One replica's parameters are a flat fp32
 * vector W1 [n1][n0], b1 [n1], W2 [n2][n1], b2 [n2], W3 [n3][n2], b3 [n3] (each W
 * row-major [out][in]); abs_mlp_param_count gives its length d.                    */
int abs_mlp_param_count(const int* dims, long long* out);
/* Bytes of scratch abs_mlp_grads needs for M workers and batch size b. */
int abs_mlp_scratch_bytes(int M, long long b, const int* dims, size_t* out);

/* Forward and backward pass of all M workers on their batches (Algorithm 2,
 * local batch gradient step): writes the batch gradients Gb [M][d] and
 * leaves activations and deltas in `scratch` (device, caller-owned) for
 * abs_mlp_per_sample.  inputs [n][n0] fp32, labels [n] int32, idx [M][idx_stride]
 * int32 sample indices (first b used), X [M][d] parameters (replica stride d).     */
int abs_mlp_grads(abs_ctx* ctx, const float* inputs, const int* labels, long long n, const int* dims,
                  const int* idx, long long idx_stride, const float* X, int M, long long b,
                  float* Gb, void* scratch, size_t scratch_bytes, void* stream);

/* Per-sample gradients of one worker as rows G [b][row_stride] (row_stride >= d; a
 * multiple of 4 keeps the rows 16-byte aligned for the fast statistics kernels),
 * from the scratch a preceding abs_mlp_grads call with the same b filled
 * (Algorithm 1, per-sample gradient step).  b <= 65535.                       */
int abs_mlp_per_sample(abs_ctx* ctx, const int* dims, long long b, int worker, const void* scratch,
                       float* G, long long row_stride, void* stream);

/* The statistics of all M workers without forming the per-sample gradient matrix
 * (a per-sample gradient of a layer is the outer product delta_i (x) h_i, so
 * ||g_i||^2 = sum_l ||delta_l,i||^2 (||h_{l-1},i||^2 + 1) and
 * <g_i, gbar> = sum_l delta_l,i^T (dW_l h_{l-1},i + db_l); Eq. def_var expanded):
 * reads the activations and deltas a preceding abs_mlp_grads call with the same b
 * and M left in `scratch` and the batch gradients Gb [M][d] it wrote; writes
 * stats [M].  The expansion sum_i ||g_i||^2 - b N loses accuracy only when the
 * variance is far below b N, i.e. when the test is satisfied by a wide margin.      */
int abs_mlp_fused_stats(abs_ctx* ctx, const int* dims, long long b, int M, void* scratch,
                        size_t scratch_bytes, const float* Gb, abs_stats* stats, void* stream);

/* One communication round of local SGD on the MLP problem, as abs_logreg_round.  At
 * the last local step the statistics come either from per-sample gradients
 * materialised for one worker at a time in G_scratch [b][g_row_stride], or, when
 * G_scratch is NULL, from abs_mlp_fused_stats.  Gb_scratch [M][d].                  */
int abs_mlp_round(abs_ctx* ctx, const float* inputs, const int* labels, long long n, const int* dims,
                  const int* idx, long long idx_stride, float* X, int M, int H, long long b, float lr,
                  const abs_test_cfg* cfg, void* scratch, size_t scratch_bytes, float* G_scratch,
                  long long g_row_stride, float* Gb_scratch, abs_stats* stats, long long* T_out,
                  long long* b_dev, abs_round_ctl* ctl, void* stream);

/* The MLP round with the test after every local step, as abs_logreg_round_per_step; the
 * statistics of every step come from abs_mlp_fused_stats.  scratch must hold M workers at
 * b_max (abs_mlp_scratch_bytes).  Waits for the stream once per local step.              */
int abs_mlp_round_per_step(abs_ctx* ctx, const float* inputs, const int* labels, long long n,
                           const int* dims, const int* idx, long long idx_stride, float* X, int M,
                           int H, long long* b_host, float lr, const abs_test_cfg* cfg,
                           const abs_round_opts* opts, void* scratch, size_t scratch_bytes,
                           float* Gb_scratch, abs_stats* stats, long long* T_out, long long* b_dev,
                           void* stream);

#ifdef __cplusplus
}
#endif
#endif  /* ABS_H_ */
