/*
 * cdgrab.h -- C ABI of the B200 (sm_100a) PairBalance ordering library for CD-GraB
 * (Coordinated Distributed Gradient Balancing, arXiv 2302.00845).
 *
 * The library plays the paper's order server for m logical workers simulated on one
 * GPU.  Per epoch it keeps one running sum r in R^d; per step it receives, for every
 * worker, the two stale gradients of the next pair of its current order, balances the m
 * pair differences against r in worker order, and records where each pair's two items go
 * in that worker's next-epoch permutation.  Algorithms are numbered by order of
 * appearance in the paper: 1 reorder by balanced signs, 2 PairBalance, 3 workers,
 * 4 parameter server, 5 probabilistic balancing, 6 balancing without normalization,
 * 7 server-side PairBalance over a set of vectors.
 *
 * Conventions
 *   - Every pointer argument says whether it is a DEVICE or a HOST pointer.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     Calls that take a stream only enqueue work; they do not synchronise the host.
 *   - All device work of one handle must be issued on one stream (or on streams the
 *     caller orders itself).  One handle is used by one host thread at a time.
 *   - The library's kernels are chained with programmatic dependent launch and the last
 *     kernel of a step lets its dependents be scheduled early.  Ordinary launches, copies
 *     and events after a library call are ordered as usual; a caller's kernel that is itself
 *     launched with programmatic stream serialization directly after a library call must
 *     execute griddepcontrol.wait (cudaGridDependencySynchronize) before it touches anything
 *     the call reads or writes.
 *   - Return value: CDGRAB_OK (0) or a negative CDGRAB_ERR_* code.  Argument and state
 *     errors leave the handle unchanged.  Conditions found on the device (non-finite
 *     reductions, an expired bounded wait) are written to a device status word and
 *     reported by cdgrab_status().
 *   - The library owns r, both permutation buffers, the sign/margin records and all
 *     scratch; they are allocated once in cdgrab_create and nothing is allocated per
 *     step.  The caller owns every buffer it passes in.
 *   - There is no CPU fallback: without a CUDA device of compute capability 10.x the
 *     create call fails.
 */
#ifndef CDGRAB_H_
#define CDGRAB_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct cdgrab_ctx cdgrab_t; /* opaque, library-owned */

enum { CDGRAB_F32 = 0, CDGRAB_BF16 = 1 };

enum {
  CDGRAB_OK = 0,
  CDGRAB_ERR_INVALID = -1,   /* bad m/n/d/dtype, NULL pointer, odd n, misaligned buffer  */
  CDGRAB_ERR_STATE = -2,     /* step outside an epoch, more than n/2 steps, early end    */
  CDGRAB_ERR_CUDA = -3,      /* a CUDA runtime/driver call failed                        */
  CDGRAB_ERR_NOMEM = -4,     /* device or host allocation failed                         */
  CDGRAB_ERR_NONFINITE = -5, /* NaN/Inf met in a reduction (device status word)          */
  CDGRAB_ERR_TIMEOUT = -6,   /* a bounded device-side wait expired (device status word)  */
  CDGRAB_ERR_DEVICE = -7,    /* no usable sm_100 device                                  */
  CDGRAB_ERR_TOO_LARGE = -8, /* size beyond the fixed scratch of cdgrab_step_noalloc        */
  CDGRAB_ERR_CORRUPT = -9    /* debug build only: guard bytes around library memory were
                                overwritten, or an index check in a kernel failed            */
};

/* Which code path a handle uses (cdgrab_path / CDGRAB_FORCE_PATH). */
enum {
  CDGRAB_PATH_AUTO = 0,
  CDGRAB_PATH_FUSED = 1, /* one launch per step, whole step on chip (small d)            */
  CDGRAB_PATH_FMA = 2,   /* two passes, Gram matrix on the fp32 FMA pipe                 */
  CDGRAB_PATH_UMMA = 3,  /* two passes, Gram matrix on tcgen05 tensor cores (bf16)       */
  CDGRAB_PATH_INDEPENDENT = 4, /* ID-GraB mode: one running sum per worker (see below)    */
  CDGRAB_PATH_LITERAL = 5 /* one launch per step, Algorithm 6 worker by worker (short rows) */
};

/*
 * Create an order-server state for m workers with n items each (n even; the paper takes
 * n even without loss of generality, Appendix B.1, and gives no rule for an unpaired
 * item, so odd n is CDGRAB_ERR_INVALID) and gradients of dimension d stored as `dtype`.
 * The current permutation of every worker starts as the identity (the paper leaves the
 * initial permutations open, Algorithm 4).  Uses the CUDA device current at the call.
 * Limits: 1 <= m <= 1024, 2 <= n, 1 <= d, m*n < 2^31.
 * On success *out receives the handle.
 */
int cdgrab_create(int m, int n, long long d, int dtype, cdgrab_t **out);

/*
 * Same interface for ID-GraB (PairBal), the uncoordinated baseline of the paper's experiments
 * (Section 5): every worker i keeps its own running sum r_i and balances its own differences
 * against it, s_i = +1 iff <r_i, c_i> < 0, r_i <- r_i + s_i c_i; the workers do not see each
 * other.  Equals m separate handles with m = 1.  The handle holds m*d floats of running sums.
 * cdgrab_get_r returns worker 0's sum, cdgrab_get_r_worker any worker's; margins are
 * |<r_i,c_i>| / (||r_i|| ||c_i||) computed directly.  cdgrab_step_randomized and
 * cdgrab_step_mean are CDGRAB_ERR_INVALID on such a handle.
 */
int cdgrab_create_independent(int m, int n, long long d, int dtype, cdgrab_t **out);

/* Running sum of one worker of an independent-mode handle: out is HOST or DEVICE float [d]. */
int cdgrab_get_r_worker(cdgrab_t *h, int worker, float *out, void *stream);

/*
 * Column-sharded order server (the direction the paper's conclusion calls an order server; the
 * method reduces over d, so it shards over d with one small exchange per step).  Each shard -- a
 * GPU, or a slice on one GPU -- owns d_local consecutive columns of every gradient row and of r.
 * Per step:
 *   cdgrab_step_begin  (every shard)  pass 1 over the shard's columns; its partial G = C^T C and
 *                      b = C^T r land in gram_out_dev: DEVICE double [m*m + m], caller-owned
 *   the caller sums those m*m + m doubles over all shards (e.g. one NCCL all-reduce) so that
 *   every shard holds the same totals
 *   cdgrab_step_finish (every shard)  the m decisions of Algorithm 6 on the totals -- identical on
 *                      every shard -- then the update of the shard's slice of r
 * grads_dev is the shard's slice [2][m][d_local] (contiguous), the same buffer in both calls.
 * All other calls (begin/end_epoch, get_*, set_perms) work as usual on each shard; signs and
 * permutations come out identical everywhere.  cdgrab_step itself, the randomized rule and the
 * fused average are not available on a shard handle.
 */
int cdgrab_create_shard(int m, int n, long long d_local, int dtype, cdgrab_t **out);
int cdgrab_step_begin(cdgrab_t *h, const void *grads_dev, double *gram_out_dev, void *stream);
int cdgrab_step_finish(cdgrab_t *h, const void *grads_dev, const double *gram_in_dev, void *stream);

/* Free the handle and everything it owns.  Synchronises the device.  NULL is allowed. */
int cdgrab_destroy(cdgrab_t *h);

/*
 * Replace the current permutations before an epoch is opened (Algorithm 4, "send initial
 * permutations").  perms_in: HOST or DEVICE pointer, int32 [m][n], every row a permutation
 * of 0..n-1 (validated on the host; anything else is CDGRAB_ERR_INVALID).  Synchronous.
 */
int cdgrab_set_perms(cdgrab_t *h, const int32_t *perms_in);

/*
 * Open an epoch: r <- 0, pair counter <- 0, sign list emptied (Algorithm 4, first line of
 * the epoch loop).  Asynchronous on `stream`.  CDGRAB_ERR_STATE if an epoch is open.
 */
int cdgrab_begin_epoch(cdgrab_t *h, void *stream);

/*
 * One balancing step: pair index k = number of steps so far in this epoch.
 *
 * grads_dev: DEVICE pointer, `dtype` elements, layout [2][m][d] contiguous, 16-byte
 *   aligned.  Slab 0 row i is the stale gradient worker i produced at position 2k of its
 *   current order (z1 of Algorithm 2), slab 1 row i the one at position 2k+1 (z2): two
 *   consecutive gather buffers of the server (Algorithm 4).  Must stay valid and unchanged
 *   until the work this call enqueued on `stream` has completed.
 *
 * Computes, for i = 0..m-1 in this order (Algorithm 7's inner loop): c_i = z1_i - z2_i;
 * s_i = +1 if ||r + c_i||_2 < ||r - c_i||_2, i.e. <r,c_i> < 0, else -1 (Algorithm 6; a
 * tie gives -1); r <- r + s_i c_i; and writes the front slot k and the back slot n-1-k of
 * worker i's next permutation: the item that received +1 goes to the front, the other to
 * the back (Algorithm 7's pointer updates, equal to Algorithm 1's list form).
 * r is kept in fp32; reductions accumulate in fp32 partial sums combined in fp64.
 *
 * Asynchronous on `stream`.  CDGRAB_ERR_STATE outside an epoch or after n/2 steps.
 */
int cdgrab_step(cdgrab_t *h, const void *grads_dev, void *stream);

/*
 * cdgrab_step with the randomized balance rule the paper's theory is stated for
 * (RandomizedBalance, the subroutine of Algorithm 2, with the bound w of Algorithm 5 made
 * explicit; Algorithm 2 prints w = 1): for worker i, p_i = 1/2 - <r,c_i>/(2w) and s_i = +1 with
 * probability p_i.  The draws are the caller's: s_i = +1 iff u_dev[i] < p_i.
 *   u_dev: DEVICE float [m], uniforms in [0,1), must stay valid until the step's work completes
 *   w:     bound, w > 0 (else CDGRAB_ERR_INVALID)
 * Where |<r,c_i>| > w Algorithm 5 would stop; here p_i leaves [0,1], the decision becomes the
 * greedy one, and the position is counted (cdgrab_out_of_bound).  Algorithm 5's other stopping
 * condition, ||r||_inf > w, is not evaluated.  Everything else is as in cdgrab_step.
 */
int cdgrab_step_randomized(cdgrab_t *h, const void *grads_dev, const float *u_dev, double w, void *stream);

/*
 * The same rule with the draws made by the library, so that a randomized epoch can be repeated
 * from (seed, epoch) alone: u_i for worker i at the handle's current pair index k is the top 24
 * bits, times 2^-24, of the first output word of Philox4x32-10 (Salmon et al., SC 2011) with the
 * key (low, high half of seed) and the counter (i, k, epoch, 0).  The caller says which epoch it
 * is in.  cdgrab_randomized_uniforms writes the m draws of (seed, epoch, k) to u_out_dev (DEVICE
 * float [m]) without touching a handle.  Errors as for cdgrab_step_randomized.
 */
int cdgrab_step_randomized_seeded(cdgrab_t *h, const void *grads_dev, unsigned long long seed, unsigned epoch,
                                  double w, void *stream);
int cdgrab_randomized_uniforms(unsigned long long seed, unsigned epoch, unsigned k, int m, float *u_out_dev,
                               void *stream);

/* Synchronise the device and return how many positions of the current/last epoch had
 * |<r,c>| > w under the randomized rule (negative CDGRAB_ERR_* on error). */
long long cdgrab_out_of_bound(cdgrab_t *h);

/*
 * cdgrab_step that also returns what the paper's parameter server sends back to the workers
 * (Algorithm 4, "compute avg. gradient ... send to all the workers"): the average of each of
 * the two gather buffers, mean_out_dev[q][x] = (1/m) sum_i grads_dev[q][i][x] for q = 0, 1.
 * mean_out_dev: DEVICE float [2][d], 16-byte aligned, caller-owned.  The rows are summed in
 * fp32 in worker order while pass 2 has them in registers, so the average costs no extra read
 * of the inputs.  Otherwise identical to cdgrab_step (same errors, same asynchrony).
 */
int cdgrab_step_mean(cdgrab_t *h, const void *grads_dev, float *mean_out_dev, void *stream);

/*
 * `count` consecutive steps of Algorithm 7's outer loop in one call, for gradients that are
 * staged ahead (a whole epoch of a small problem): grads_dev is DEVICE memory laid out
 * [count][2][m][d] in the handle's dtype, 16-byte aligned, step j at offset j*2*m*d elements.
 * The result is bit-identical to `count` calls of cdgrab_step on the slices (greedy rule of
 * Algorithm 6).  On the single-launch paths (small steps) the steps run inside one kernel launch
 * and the running sum never leaves the SM between them; on the other paths the call
 * loops over cdgrab_step.  With the environment variable CDGRAB_DEFER=1 at create time, handles
 * on the two-pass FMA path with long rows (m <= 16, d >= 65536) instead let pass 1 of step j
 * apply the running-sum update of step j-1 (Algorithm 6's r <- r + s c, deferred by one step):
 * count + 1 streaming launches and one read of r per step, same bits; measured slower than the
 * loop, hence off by default.  CDGRAB_ERR_STATE if fewer than `count` steps remain in the epoch
 * (nothing is done then); CDGRAB_ERR_INVALID on a shard handle or count < 1.  Asynchronous on
 * `stream` like cdgrab_step.
 */
int cdgrab_step_many(cdgrab_t *h, const void *grads_dev, int count, void *stream);

/*
 * Close the epoch after exactly n/2 steps (else CDGRAB_ERR_STATE): the next permutations
 * become the current ones (Algorithm 4, last lines of the epoch loop) and, if perms_out is
 * not NULL, are copied there.  perms_out: HOST or DEVICE pointer, int32 [m][n];
 * perms_out[i][j] = item worker i visits at position j in the next epoch.  The copy is
 * enqueued on `stream` (pageable host memory makes it synchronous).
 */
int cdgrab_end_epoch(cdgrab_t *h, int32_t *perms_out, void *stream);

/* ---- read-back helpers (no semantics of their own; the parity tests need them) ------ */

/* Signs of the current/last epoch: out is HOST or DEVICE int8 [m][n/2], +1/-1, 0 where no
 * step has been taken yet.  Enqueued on `stream`. */
int cdgrab_get_signs(cdgrab_t *h, int8_t *out, void *stream);

/* Running sum: out is HOST or DEVICE float [d].  Enqueued on `stream`. */
int cdgrab_get_r(cdgrab_t *h, float *out, void *stream);

/* Relative margins |<r,c>| / (||r|| ||c||) seen at each decision (0 when r = 0 or c = 0):
 * out is HOST or DEVICE float [m][n/2].  ||r||^2 is tracked by the recurrence
 * ||r + s c||^2 = ||r||^2 + 2 s <r,c> + ||c||^2.  Enqueued on `stream`. */
int cdgrab_get_margins(cdgrab_t *h, float *out, void *stream);

/* Current permutations: out is HOST or DEVICE int32 [m][n].  Enqueued on `stream`. */
int cdgrab_get_perms(cdgrab_t *h, int32_t *out, void *stream);

/* Next-epoch permutations as far as the open epoch has filled them (front slots 0..k-1 and
 * back slots n-k..n-1 of every worker; other slots hold stale values): out is HOST or DEVICE
 * int32 [m][n].  Enqueued on `stream`. */
int cdgrab_get_next_perms(cdgrab_t *h, int32_t *out, void *stream);

/* Synchronise the device and return the first device-side condition recorded since
 * creation (CDGRAB_ERR_NONFINITE, CDGRAB_ERR_TIMEOUT, CDGRAB_ERR_CUDA) or CDGRAB_OK. */
int cdgrab_status(cdgrab_t *h);

/* Synchronise the device and clear the device status word (after the caller has dealt with a
 * reported condition). */
int cdgrab_clear_status(cdgrab_t *h);

/*
 * Self-test of the bounded device-side wait used by the TMA-fed kernels: a one-thread kernel
 * waits on a barrier that nothing completes, gives up after `cycles` SM clock cycles
 * (1 .. 2e9), raises the time-out bit of the status word and returns; nothing is in flight, so
 * the context stays usable.  Synchronous.  *waited_cycles (HOST, may be NULL) receives how long
 * the kernel actually waited.  Afterwards cdgrab_status() reports CDGRAB_ERR_TIMEOUT until
 * cdgrab_clear_status() is called.
 */
int cdgrab_selftest_wait_timeout(cdgrab_t *h, long long cycles, long long *waited_cycles);

/*
 * Checkpoint / resume.  cdgrab_save_state copies everything a handle needs to continue (epoch
 * position, running sum(s), both permutation tables, signs, margins) into host_buf (HOST, at
 * least cdgrab_state_bytes(h) bytes); cdgrab_load_state puts it into a handle created with the
 * same m, n, d, dtype and mode (else CDGRAB_ERR_INVALID), in or between epochs.  Both are
 * synchronous.  A run continued from a loaded state gives bit-identical results.
 */
long long cdgrab_state_bytes(const cdgrab_t *h);
int cdgrab_save_state(cdgrab_t *h, void *host_buf, long long bytes);
int cdgrab_load_state(cdgrab_t *h, const void *host_buf, long long bytes);

/* Code path the handle uses (CDGRAB_PATH_*).  The environment variable
 * CDGRAB_FORCE_PATH = fused | fma | umma | literal, read at create time, overrides the automatic
 * choice when the forced path supports the shape; otherwise create fails with
 * CDGRAB_ERR_INVALID. */
int cdgrab_path(const cdgrab_t *h);

/* Number of kernels the library has launched through this handle so far. */
long long cdgrab_launch_count(const cdgrab_t *h);

/* Kernel kinds for the timing hook below. */
enum {
  CDGRAB_K_GRAM = 0,    /* pass 1: Gram matrix G = C^T C and b = C^T r                    */
  CDGRAB_K_COMBINE = 1, /* fixed-order fp64 sum of pass-1 partials                        */
  CDGRAB_K_SCAN = 2,    /* the m sign decisions + permutation slots                       */
  CDGRAB_K_UPDATE = 3,  /* pass 2: r <- r + sum_i s_i c_i                                 */
  CDGRAB_K_FUSED = 4,   /* whole step in one launch                                       */
  CDGRAB_K_LOGREG = 5,  /* per-example logistic-regression gradients                      */
  CDGRAB_K_COUNT = 6
};

/* Timing hook: while on, every kernel the handle launches is bracketed by a pair of CUDA
 * events recorded on the launching stream (at most 8192 launches are kept; later ones are
 * not recorded).  Turning it on clears earlier records.  Costs two event records per launch. */
int cdgrab_profile_enable(cdgrab_t *h, int on);

/* Synchronise the device and report, for kernel kind `kind`, the summed event-to-event
 * duration in milliseconds and the number of recorded launches.  HOST pointers. */
int cdgrab_profile_read(cdgrab_t *h, int kind, double *total_ms, long long *launches);

/* Static message for a CDGRAB_* code. */
const char *cdgrab_strerror(int code);

/*
 * Per-example logistic-regression gradients for the current step (the workers' gradient
 * computation of Algorithm 3 for the logistic-regression task of Section 5), written in
 * the layout cdgrab_step consumes.  For worker i and slot q in {0,1}: item
 * j = perm_cur[i][2k+q], z = <w, X[i][j]>, g = (1/(1+exp(-z)) - y[i][j]) * X[i][j].
 *   X: DEVICE float [m][n][d]; y: DEVICE float [m][n] with values in {0,1};
 *   w: DEVICE float [d]; grads_out: DEVICE float [2][m][d].  Handle dtype must be F32.
 * Asynchronous on `stream`.
 */
int cdgrab_logreg_grads(cdgrab_t *h, const float *X, const float *y, const float *w,
                        float *grads_out, void *stream);

/*
 * Logistic regression without a gradient buffer: cdgrab_logreg_grads followed by cdgrab_step in
 * one launch, the pair differences formed straight from the feature rows,
 *   c_i = (sigma(<w,x_p>) - y_p) x_p - (sigma(<w,x_q>) - y_q) x_q,  p, q = perm_cur[i][2k], [2k+1]
 * (each product rounded to fp32 as a stored gradient would be).  Same arguments as
 * cdgrab_logreg_grads minus the output; X and w 16-byte aligned.  Only for fp32 handles small
 * enough for a single-launch path (cdgrab_path == CDGRAB_PATH_FUSED, or CDGRAB_PATH_LITERAL with
 * m <= 16), else CDGRAB_ERR_INVALID.
 * Counts as one balancing step.  Asynchronous on `stream`.
 */
int cdgrab_step_logreg(cdgrab_t *h, const float *X, const float *y, const float *w, void *stream);

/*
 * Same step with the gradients in HOST memory (pinned memory makes the copy
 * asynchronous): grads_host [2][m][d] is copied into staging_dev (DEVICE, at least
 * 2*m*d elements, 16-byte aligned, caller-owned) on `stream`, then cdgrab_step runs on it.
 */
int cdgrab_step_host(cdgrab_t *h, const void *grads_host, void *staging_dev, void *stream);

/*
 * Parallel herding objective, Eq. (7) of the paper -- the bound PairBalance is meant to shrink:
 *   max over k in [n] of || sum_{j<=k} sum_{i<m} ( z[i][perms[i][j]] - zbar ) ||_inf ,
 * zbar = mean of all m*n vectors.  Stand-alone (no handle), fp64 sums in a fixed order.
 *   z_dev      DEVICE float [m][n][d], vectors indexed by item id
 *   perms_dev  DEVICE int32 [m][n], row i = the order in which worker i visits its items
 *   workspace_dev  DEVICE, 8-byte aligned, at least cdgrab_herding_workspace_bytes(m, n, d) bytes,
 *              caller-owned scratch (contents undefined afterwards)
 *   out_dev    DEVICE double [1], receives the objective
 * Asynchronous on `stream`.  CDGRAB_ERR_INVALID for NULL pointers, non-positive sizes, a
 * workspace that is too small or misaligned.
 */
long long cdgrab_herding_workspace_bytes(int m, int n, long long d);
int cdgrab_herding_objective(const float *z_dev, const int32_t *perms_dev, int m, int n, long long d,
                             void *workspace_dev, long long workspace_bytes, double *out_dev, void *stream);

/*
 * One balancing step that allocates nothing (the paper has no counterpart: this is a
 * packaging of cdgrab_step for a restricted kind of caller).
 *
 * Some callers cannot call cudaMalloc: plug-ins that are handed buffers and a stream and
 * nothing else, code inside a framework's caching allocator whose pool a raw allocation
 * would fragment or overrun, loops that cannot afford the device-wide synchronisation an
 * allocation or a free implies.  They cannot use cdgrab_create either.  This call keeps no
 * handle: the caller owns the running sum and the signs, and the scratch of the two-pass
 * formulation (block partial sums, Gram matrix, a few bookkeeping words) lives in one fixed
 * array of 625,152 bytes in the library's device image, which every GPU that loads the
 * library holds until the process exits.
 *
 *   m          workers, 1 <= m <= 16; more is CDGRAB_ERR_TOO_LARGE (the fixed scratch and the
 *              register-resident kernels behind this call stop there)
 *   d          gradient dimension, a multiple of 4, d >= 4 (else CDGRAB_ERR_INVALID)
 *   dtype      CDGRAB_F32 or CDGRAB_BF16
 *   grads_dev  DEVICE, [2][m][d] as for cdgrab_step, 16-byte aligned, caller-owned
 *   r_dev      DEVICE, float [d], 16-byte aligned, caller-owned: the running sum, read and
 *              updated in place (zero it yourself at the start of an epoch)
 *   signs_out_dev  DEVICE, int8 [m], caller-owned: receives the m signs of this step
 *
 * Same arithmetic as cdgrab_step on the FMA path: for i = 0..m-1, s_i = +1 iff <r,c_i> < 0
 * with c_i = z1_i - z2_i, then r <- r + s_i c_i.  The caller applies the signs to its own
 * permutations (item with +1 to the front slot, the other to the back slot).
 *
 * The first call on a device resolves the scratch array's device address and writes its
 * constant part; that call is synchronous and should be made before any stream capture is
 * begun.  Later calls only enqueue work on `stream`.  No call allocates or frees memory.
 * All calls on a device share the scratch, which keeps the previous call's contents; the
 * words that must start at zero are cleared on `stream` at every call.  Two calls whose
 * device work may overlap (different streams without ordering, or several host threads)
 * race on the scratch: order them.
 *
 * Device-side conditions (a NaN/Inf met in a reduction) are recorded in a status word inside
 * the scratch; it stays set over later calls until cdgrab_noalloc_status reads it.
 */
int cdgrab_step_noalloc(int m, long long d, int dtype, const void *grads_dev, float *r_dev,
                        int8_t *signs_out_dev, void *stream);

/* What the kernels of cdgrab_step_noalloc reported on the current device since the last call of
 * this function (the paper has no counterpart): CDGRAB_OK, CDGRAB_ERR_NONFINITE or
 * CDGRAB_ERR_TIMEOUT.  Synchronises the device, copies one word out of the fixed scratch and
 * clears it when set; allocates nothing.  CDGRAB_OK when no step has run on this device yet.
 * Not to be called while a stream capture is open (it synchronises). */
int cdgrab_noalloc_status(void);

#ifdef __cplusplus
}
#endif
#endif /* CDGRAB_H_ */
