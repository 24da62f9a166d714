/*
 * def.h -- C boundary of the B200 (sm_100a) DEF / DEF-A / EF step library.
 *
 * One optimizer step of distributed momentum SGD with random block-wise gradient
 * sparsification (RBGS) under error feedback, from "Detached Error Feedback for
 * Distributed SGD with Random Sparsification": Algorithm 1 from its error-feedback step to its update, with the
 * momentum substitution of Eq. 10, for W simulated workers (the paper's K) held as
 * the rows of [W, d] fp32 tensors on one GPU.  Per step and per worker w:
 *
 *     m'[w,j] = mu * m[w,j] + g[w,j]                          (Eq. 10)
 *     p[w,j]  = eta * m'[w,j] + e[w,j]                        (Eq. 10; Algorithm 1's error-feedback step when mu = 0)
 *     C(p)    = p on the k block coordinates {(s+i) mod d}, 0 elsewhere   (Section 1, RBGS)
 *     e'[w,j] = p[w,j] - C(p)[w,j]                            (Algorithm 1's new-error step)
 *     x[j]   -= (1/W) * sum_w C(p)[w,j]                       (Algorithm 1: ring-allreduce, update)
 *
 * The block start s is drawn once per step, the same for every worker (Section 1:
 * all workers hold the same seed), by a counter-based Philox4x32-10 generator keyed
 * by (seed, step).  The sum over workers stands in for the algorithm's ring-allreduce;
 * it runs over w = 0..W-1 in that order in fp32, followed by an IEEE division by W.
 * Every product-and-add above is one fused multiply-add (one rounding).
 *
 * EF, DEF and DEF-A run the same step: they differ in where the caller evaluates
 * the gradient (Algorithm 1's detach step: at x_t - lambda e_{k,t}, lambda = 0 for EF) and
 * in the model that is returned after training (Algorithm 1's Output).
 *
 * Conventions
 *   - All tensors are fp32, row-major; [W, d] tensors are contiguous with row stride d
 *     unless a call takes an explicit row stride `ld` (in floats).
 *   - Pointers are DEVICE pointers on the current CUDA device unless the parameter is
 *     called *_host.  The caller owns every tensor; the library keeps no reference to
 *     them after the work it enqueued has run.
 *   - Calls that take device pointers only enqueue work on the context's stream
 *     (def_set_stream; default: the legacy default stream).  They do not synchronise
 *     and, unless a function says otherwise, allocate nothing.
 *   - Every function returns DEF_OK (0) or a negative DEF_ERR_* code and leaves a
 *     human-readable message for def_last_error() (thread-local).  Nothing is
 *     launched when validation fails.  No exception crosses this boundary.
 *   - A def_ctx is not internally locked: use it from one host thread at a time (different
 *     contexts are independent).  Work enqueued by successive calls on one stream runs in
 *     call order; tensors must stay valid until that work has run.
 *   - IEEE specials in the data propagate as the arithmetic above dictates; inputs are
 *     not scanned.
 */
#ifndef DEF_B200_H
#define DEF_B200_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct def_ctx def_ctx; /* opaque, owned by the library */

enum { DEF_VARIANT_DEF = 0, DEF_VARIANT_DEF_A = 1, DEF_VARIANT_EF = 2 };

enum {
    DEF_OK = 0,
    DEF_ERR_ARG = -1,         /* a size or hyper-parameter is out of range          */
    DEF_ERR_NULL = -2,        /* a required pointer is NULL                         */
    DEF_ERR_ALIGN = -3,       /* a pointer is not 4-byte aligned                    */
    DEF_ERR_ALIAS = -4,       /* two tensors overlap                                */
    DEF_ERR_DEVICE = -5,      /* no CUDA device, or not compute capability 10.x     */
    DEF_ERR_CUDA = -6,        /* the CUDA runtime reported an error                 */
    DEF_ERR_UNSUPPORTED = -7  /* a documented feature that is not implemented       */
};

#define DEF_MAX_WORKERS 64

/*
 * Algorithm 1's inputs.  d: model size; W: workers, 1..DEF_MAX_WORKERS; k: block
 * length, 1 <= k <= d (compression ratio d/k); variant: DEF_VARIANT_*; lr: eta,
 * finite; momentum: mu in [0, 1) (0 selects Algorithm 1's error-feedback step as printed);
 * coeffs: NULL for the defaults {0.3, 0}, else coeffs[0] = lambda in [0, 1] (the
 * detach coefficient; forced to 0 for DEF_VARIANT_EF) and coeffs[1] = weight decay,
 * which must be 0 (the paper does not say where weight decay enters: fold it into
 * the gradients; non-zero returns NULL with DEF_ERR_UNSUPPORTED).
 * Returns NULL on failure (see def_last_error).  Touches no GPU: the device is
 * checked by the first call that launches.
 */
def_ctx *def_create(int64_t d, int32_t W, int64_t k, int32_t variant, float lr, float momentum,
                    const float *coeffs);

/* Frees the handle and any device staging memory def_step_host allocated for it. */
int def_destroy(def_ctx *ctx);

/*
 * One step (Algorithm 1 from its error-feedback step to its update, Eq. 10), in place.
 *   params [d]     x_t      -> x_{t+1}   (only the k block coordinates are touched)
 *   grads  [W, d]  g_{k,t}     read only
 *   errors [W, d]  e_{k,t}  -> e_{k,t+1}
 *   mom    [W, d]  m_{k,t}  -> m_{k,t+1}; NULL if and only if momentum == 0
 *   step, seed     t and the shared seed: the block start is a pure function of both
 * The caller zeroes errors and mom before step 0 (Algorithm 1's initialisation).
 * 16-byte aligned base pointers run on 128-bit accesses whatever d is (when d % 4 != 0 the
 * rows themselves are unaligned and the contiguous [W, d] tensors are streamed flat, within 1 %
 * of the aligned speed at compression ratios of 32 and more, 3 % slower at ratio 8, where the
 * block coordinates' 4-byte accesses weigh more); bases that are only 8- or 4-byte aligned are
 * accepted and run on narrower accesses, 6 % and 14 % slower at large sizes.
 * Errors: DEF_ERR_NULL, DEF_ERR_ALIGN, DEF_ERR_ALIAS (any two of the four tensors
 * overlap), DEF_ERR_DEVICE, DEF_ERR_CUDA (launch failure).
 */
int def_step(def_ctx *ctx, float *params, const float *grads, float *errors, float *mom,
             uint64_t step, uint64_t seed);

/*
 * The same step on a contiguous range of coordinates [j0, j0 + n) of the
 * d-dimensional problem: every operation of the step is separate per coordinate, so
 * a model can be cut by columns across GPUs, or streamed through the GPU in pieces,
 * with no exchange between the pieces.  params points at the n local coordinates;
 * grads / errors / mom point at local [W, n] tensors with row stride ld >= n floats.
 * The block start is still drawn over the whole d.  0 <= j0, j0 + n <= d; n = 0 is a no-op
 * (pointers are then not looked at).
 */
int def_step_columns(def_ctx *ctx, int64_t j0, int64_t n, int64_t ld, float *params,
                     const float *grads, float *errors, float *mom, uint64_t step,
                     uint64_t seed);

/*
 * def_step / def_step_columns that also write where each worker evaluates its NEXT gradient
 * (Algorithm 1's detach step of iteration t + 1), fused into the same two kernels:
 *     detached_out[w, j] = x_{t+1}[j] - lambda * e_{w,t+1}[j]      (one fused multiply-add)
 * This is the one thing that makes DEF differ from plain EF at run time (EF, lambda = 0,
 * evaluates at x_{t+1} itself and has no use for it).  It costs one more [W, d] write:
 * 24 instead of 20 bytes per gradient element.  detached_out [W, ld] must overlap none of
 * the other tensors.  Other arguments and errors as for def_step / def_step_columns.
 * Contiguous rows with d % 4 != 0 (16-byte aligned bases, params included) keep 128-bit accesses
 * here too, 2-4 % behind rows padded to a multiple of 4 floats (ld = 4 * ceil(d / 4)).
 */
int def_step_detach(def_ctx *ctx, float *params, const float *grads, float *errors, float *mom,
                    float *detached_out, uint64_t step, uint64_t seed);
int def_step_columns_detach(def_ctx *ctx, int64_t j0, int64_t n, int64_t ld, float *params,
                            const float *grads, float *errors, float *mom, float *detached_out,
                            uint64_t step, uint64_t seed);

/*
 * The step with the WORKERS cut across GPUs (the paper's own deployment: one process per
 * GPU, each holding some of the K workers and a replica of the model; Algorithm 1's ring-allreduce step is
 * then a real all-reduce).  A context made with W = the number of LOCAL workers runs the step
 * in two halves around the caller's all-reduce:
 *   def_step_rows_local  the error-feedback and new-error steps (Eq. 10) for the local rows, in place as in def_step, and
 *                        block_sum_out[i] = sum over the local workers (in order) of C(p_w) at
 *                        block coordinate (s + i) mod d, i = 0..k-1: the k floats that travel.
 *                        params is not needed.
 *   (caller)             all-reduce(sum) of block_sum_out over the ranks -- additivity of the
 *                        compressor (Assumption 3) is what makes a plain sum valid.
 *   def_step_rows_apply  the update: params[(s + i) mod d] -= block_sum[i] / W_total.
 * Every rank passes the same (step, seed) and so cuts the same block.  With one rank the
 * result equals def_step bit for bit; with several, the order in which the all-reduce adds
 * the ranks' partial sums is the library's, so floats agree to rounding, not bitwise.
 * RBGS only (DEF_ERR_UNSUPPORTED under DEF_COMPRESSOR_SCALE).  Whole model (n = ld = d); any d
 * (16-byte aligned bases keep 128-bit accesses when d % 4 != 0, as in def_step).
 */
int def_step_rows_local(def_ctx *ctx, const float *grads, float *errors, float *mom,
                        float *block_sum_out, uint64_t step, uint64_t seed);
int def_step_rows_apply(def_ctx *ctx, float *params, const float *block_sum, int32_t W_total,
                        uint64_t step, uint64_t seed);

/*
 * The row-sharded step that also writes where each LOCAL worker evaluates its next gradient
 * (Algorithm 1's detach step of iteration t + 1; see def_step_detach), still at one extra
 * [W, d] write.  Outside the block x does not change in this step, so the local half already
 * knows z[w, j] = x_t[j] - lambda * e_{w,t+1}[j]; it reads params [d] for that and does not
 * write it.  On the k block coordinates e_{w,t+1} = +0, so z[w, j] = x_{t+1}[j], which exists
 * only after the all-reduce: the local half leaves x_t[j] there and def_step_rows_apply_detach
 * overwrites those k floats of every local row when it updates params.  After the pair of
 * calls detached_out [W, d] equals what def_step_detach would have written for these workers.
 * detached_out must overlap none of the other tensors.
 */
int def_step_rows_local_detach(def_ctx *ctx, const float *params, const float *grads, float *errors,
                               float *mom, float *block_sum_out, float *detached_out, uint64_t step,
                               uint64_t seed);
int def_step_rows_apply_detach(def_ctx *ctx, float *params, const float *block_sum, int32_t W_total,
                               float *detached_out, uint64_t step, uint64_t seed);

/*
 * Takes the all-reduce of a row-sharded step off the critical path.  The k block sums are ready
 * as soon as the few tiles that touch the block are done, long before the rest of the [W, d]
 * tensors has been streamed.  With a side stream set (a cudaStream_t other than the context's
 * stream; NULL switches back), def_step_rows_local[_detach] makes the side stream wait for what
 * the context's stream holds so far, runs the kernel of the block tiles THERE and everything
 * else on the context's stream as before; the caller enqueues its all-reduce of block_sum_out on
 * the side stream; def_step_rows_apply[_detach] runs there too, and then makes the context's
 * stream wait for it.  The collective and the update so overlap the streaming kernel, and work
 * enqueued on the context's stream after the apply call sees the finished step.  (Steps that run
 * as a single kernel -- models under the def_set_small_step_bytes threshold, bases that are not
 * 16-byte aligned -- produce the sums on the context's stream; the side stream is then made to
 * wait for that kernel, so the same calling sequence stays correct.)  The first non-NULL call
 * creates two events.  The caller owns the stream and keeps it alive while it is set.
 */
int def_set_rows_stream(def_ctx *ctx, void *side_stream);

/*
 * One step with every tensor in HOST memory (pinned memory is much faster; pageable
 * works).  The library streams column ranges through device staging buffers it owns
 * (allocated on the first call: three slots of up to 512 MiB of rows each, less for small
 * models and when free device memory is short; freed by def_destroy): host->device copy, def_step_columns' kernel and device->host copy of
 * successive ranges overlap on three streams.  Blocks until params_host,
 * errors_host and mom_host hold the results.  Same shapes as def_step.
 */
int def_step_host(def_ctx *ctx, float *params_host, const float *grads_host, float *errors_host,
                  float *mom_host, uint64_t step, uint64_t seed);

/* def_step_columns with every tensor in host memory (same streaming as def_step_host):
 * coordinates [j0, j0 + n) of the model, local [W, n] tensors with row stride ld. */
int def_step_columns_host(def_ctx *ctx, int64_t j0, int64_t n, int64_t ld, float *params_host,
                          const float *grads_host, float *errors_host, float *mom_host,
                          uint64_t step, uint64_t seed);

/*
 * The point worker w evaluates its next gradient at (Algorithm 1's detach step):
 *     detached_out[w, j] = params[j] - lambda * errors[w, j]      (one fused multiply-add)
 * lambda is coeffs[0] of def_create (0 for DEF_VARIANT_EF, which makes every row a copy of
 * params).  View arguments as in def_step_columns: n coordinates, [W, n] tensors with row
 * stride ld; the whole model is n = ld = d.  detached_out [W, ld] must not overlap the
 * inputs (DEF_ERR_ALIAS).  Enqueued on the context's stream.
 */
int def_detach(def_ctx *ctx, int64_t n, int64_t ld, const float *params, const float *errors,
               float *detached_out);

/*
 * The model Algorithm 1 returns after training (its output line):
 *     DEF_VARIANT_DEF:            model_out[j] = params[j] - (sum_w errors[w, j]) / W
 *                                 (y_T; workers added in order w = 0..W-1 in fp32, IEEE division)
 *     DEF_VARIANT_DEF_A, _EF:     model_out = params (x_T); errors may be NULL
 * model_out [n] must not overlap the inputs.  Enqueued on the context's stream.
 */
int def_output(def_ctx *ctx, int64_t n, int64_t ld, const float *params, const float *errors,
               float *model_out);

/*
 * The squared distances the paper's analysis is about (Eq. 9 and the paragraph before it),
 * over the n coordinates of the view, accumulated in fp64 from the fp32 errors:
 *     stats_out[0] = (1/W) sum_w |e_w|^2            bound on plain EF's distance |x_t - y_t|^2
 *     stats_out[1] = |e_bar|^2, e_bar = mean_w e_w  that distance itself
 *     stats_out[2] = (1/W) sum_w |e_bar - lambda e_w|^2     Eq. 9, DEF's distance
 * stats_out[2] is formed as (1 - 2 lambda) stats_out[1] + lambda^2 stats_out[0], the same
 * quantity with the square expanded.  All three are sums over coordinates, so the results of
 * column shards add.  stats_out: 3 doubles in DEVICE memory, written on the context's stream.
 * Two kernels: per-CTA partial sums into a 32 KB scratch buffer the context owns (the first
 * call allocates it with cudaMalloc; def_destroy frees it), then one CTA adds them in a fixed
 * order, so repeated calls give identical bits.
 */
int def_stats(def_ctx *ctx, int64_t n, int64_t ld, const float *errors, double *stats_out);

/*
 * def_stats for callers that cannot allocate device memory.  (The paper has no counterpart
 * to this entry point; it exists for the integration, not for the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a framework that
 * owns all device memory through its own pool and forbids side allocations, in a real-time
 * or pre-sized deployment whose memory budget is fixed before start-up, or on a path where
 * the implicit device synchronisation of cudaMalloc / cudaFree is not acceptable.  def_stats
 * takes its 32 KB of partial-sum scratch from cudaMalloc on first use; this variant keeps the
 * same scratch in a fixed array inside the library's device image, so it never calls
 * cudaMalloc, cudaFree or any allocating routine.  Every GPU that loads the library holds
 * those 32 KB (2 * DEF_STATS_STATIC_SLOTS doubles) until the process exits.
 *
 * It computes exactly what def_stats computes, with the same kernels, and needs no def_ctx:
 * errors [W, ld] (device, fp32), n coordinates per row, W workers (1..DEF_MAX_WORKERS),
 * lambda in [0, 1], stats_out = 3 doubles in device memory, cuda_stream = a cudaStream_t
 * (NULL = legacy default stream).  The work is enqueued; nothing is synchronised.
 *
 * Limits and rules:
 *   - n <= DEF_STATS_STATIC_MAX_N per call; larger n returns DEF_ERR_ARG with a message
 *     (cut the columns into ranges and add the three results -- they are sums over
 *     coordinates -- or use def_stats).
 *   - The first call on each device looks up the array's device address (one query of the
 *     runtime's symbol table, with that device current) and remembers it.  Make that first
 *     call outside any stream capture.
 *   - All calls on a device share the one array, and it keeps whatever the last call left
 *     there.  A call overwrites every slot it later reads, so stale contents are harmless and
 *     nothing is cleared; but two calls whose kernels overlap on the GPU (different streams,
 *     or different host threads on different streams) race on it and return garbage.
 *     Serialise them: one stream, or an event between them.
 * Errors: DEF_ERR_NULL, DEF_ERR_ALIGN, DEF_ERR_ARG, DEF_ERR_DEVICE, DEF_ERR_CUDA.
 */
#define DEF_STATS_STATIC_SLOTS 2048
#define DEF_STATS_STATIC_MAX_N ((int64_t)1 << 31)
int def_stats_static(const float *errors, int64_t n, int64_t ld, int32_t W, float lambda,
                     double *stats_out, void *cuda_stream);

/* The stream device-pointer calls enqueue on (a cudaStream_t; NULL = legacy default). */
int def_set_stream(def_ctx *ctx, void *cuda_stream);

/*
 * The compressor C of the step.  DEF_COMPRESSOR_RBGS (default) is the random block of
 * Section 1 with the k given to def_create.  DEF_COMPRESSOR_SCALE is C(v) = delta * v,
 * 0 < delta < 1, the case the DEF-A paragraph uses to show that x_t becomes a geometric
 * average of the SGD iterates y_t (Eq. 11): every coordinate is sent, e' = p - delta p, and
 * params is updated everywhere; k, step and seed are then ignored.  `delta` is ignored for
 * RBGS.  Applies to every later step call of this context.
 */
enum { DEF_COMPRESSOR_RBGS = 0, DEF_COMPRESSOR_SCALE = 1 };
int def_set_compressor(def_ctx *ctx, int32_t compressor, float delta);

/*
 * Launch strategy of a step whose tensors start on 16-byte boundaries.  A step that moves at
 * least `bytes` (20 * W * n) runs as a pair of kernels (block coordinates, then everything else
 * as a stream that is allowed to start beside the first); a smaller one runs as one launch of
 * the general kernel.  Default 128 MiB: below that a step is bound by the launches themselves
 * when run back to back; 0 always uses the pair.  Results are bit-identical either way.
 */
int def_set_small_step_bytes(def_ctx *ctx, int64_t bytes);

/*
 * Whether the second kernel of a pair may start while the first (the tiles that touch the block)
 * is still running -- they write disjoint floats, and work enqueued after the pair is ordered
 * behind both either way.  DEF_OVERLAP_AUTO (default) leaves the choice to the library (side by
 * side at every size: it was at least as fast wherever it was measured), DEF_OVERLAP_NEVER runs
 * the two one after the other, DEF_OVERLAP_ALWAYS side by side.  Results are bit-identical in
 * every mode.
 */
enum { DEF_OVERLAP_AUTO = 0, DEF_OVERLAP_NEVER = 1, DEF_OVERLAP_ALWAYS = 2 };
int def_set_pair_overlap(def_ctx *ctx, int32_t mode);

/* Learning-rate schedules: eta may change between steps. */
int def_set_lr(def_ctx *ctx, float lr);

/*
 * The block start s_t in [0, d) that a step with (step, seed) uses, computed on the
 * host by the library's own Philox4x32-10: key = (seed low, seed high), counter =
 * (step low, step high, 0x52424753, 0), r = word0 | word1 << 32, s = floor(r d / 2^64).
 */
int def_block_start(const def_ctx *ctx, uint64_t step, uint64_t seed, int64_t *start_out);

/*
 * The same start computed by the device code the step kernels use, for a batch:
 * starts_out[i] = start(seeds[i], steps[i], ds[i]).  All four are device arrays of
 * n elements (uint64, uint64, int64, int64); ds[i] >= 1.  Enqueued on `cuda_stream`.
 */
int def_block_start_device(const uint64_t *seeds, const uint64_t *steps, const int64_t *ds,
                           int64_t n, int64_t *starts_out, void *cuda_stream);

/*
 * Profiling aid.  A step on 16-byte aligned rows is two kernels: DEF_KERNEL_BLOCK does the
 * tiles of 1024 coordinates that touch the block (cross-worker sum, update of params),
 * DEF_KERNEL_STREAM all the others; narrower alignments and the d % 4 tail run
 * DEF_KERNEL_GENERAL.  With timing enabled every launch is bracketed by CUDA events on the
 * context's stream and WAITED for, and its device time is added to its kernel's total:
 * calls then block, so leave it off when measuring throughput.  def_kernel_time reads the
 * totals accumulated since def_create.
 */
enum { DEF_KERNEL_STREAM = 0, DEF_KERNEL_BLOCK = 1, DEF_KERNEL_GENERAL = 2, DEF_KERNEL_KINDS = 3 };
int def_set_kernel_timing(def_ctx *ctx, int enable);
int def_kernel_time(const def_ctx *ctx, int kernel, double *total_ms_out, int64_t *launches_out);

/*
 * How a step with (step, seed) on local coordinates [j0, j0 + n) is cut between the two kernels of
 * a pair, computed on the host from the same block start the kernels draw.  Tiles are runs of 1024
 * local coordinates.  The tiles that touch the block (Section 1's k coordinates from s, wrapping
 * mod d) are tiles [0, plan_out[2]) and [plan_out[0], plan_out[0] + plan_out[1]), disjoint; the
 * block kernel gets one CTA for each, the stream kernel CTAs for the other plan_out[3] tiles.
 * n >= 1.  Touches no GPU.
 */
int def_tile_plan(const def_ctx *ctx, int64_t j0, int64_t n, uint64_t step, uint64_t seed, int64_t plan_out[4]);

/* Kernels this context has launched so far (every launch of every call). */
int def_launch_count(const def_ctx *ctx, int64_t *count_out);

/* Message of the last failure on this thread ("" if none). */
const char *def_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* DEF_B200_H */
