/*
 * regtopk.h: C ABI of the RegTop-k sparsification step for N workers batched on one GPU.
 *
 * The calls follow the paper's statement of the method (arXiv 2501.05633):
 *   - Algorithm 2 ("RegTop-k sparsification at worker n"): accumulate a = eps + g, posterior
 *     distortion Delta on the previous mask's support (Eq. (Delta_def)), score
 *     |a| * tanh(|1 + Delta| / mu), top-k mask of the score, send the raw accumulator on the mask,
 *     residual eps' = a - ghat.  Round 0, and mu == 0, are Algorithm 1 (Top-k with error
 *     accumulation).
 *   - Section 2.2: the top-k selector and the server aggregation g = sum_n omega_n * ghat_n.
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer unless its comment says "host".
 *   - The caller owns every buffer it passes, including the workspace; the library allocates no
 *     device memory.  It owns only a small host-side context (malloc'ed by regtopk_create, freed by
 *     regtopk_destroy).
 *   - Calls enqueue work on the CUDA stream given at creation and return without synchronising,
 *     except where stated.  Buffers must stay valid until that work has run.
 *   - Return value: REGTOPK_OK (0) or a negative REGTOPK_ERR_* code.  Nothing aborts, throws or traps.
 *   - Arithmetic: binary32, every operation individually rounded in the written order (no fused
 *     multiply-add), so results are reproducible bit for bit; selection is exact, ties between equal
 *     scores go to the lower index.  Gradients must be finite.
 *   - One GPU, one context per (d, N, k) problem; contexts are independent.  A context is not
 *     thread-safe.
 */
#ifndef REGTOPK_H_
#define REGTOPK_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct regtopk_ctx regtopk_ctx;

enum {
  REGTOPK_OK = 0,
  REGTOPK_ERR_INVALID_ARG = -1,         /* a size, pointer, alignment or hyper-parameter is unusable   */
  REGTOPK_ERR_WORKSPACE_TOO_SMALL = -2, /* workspace_bytes < regtopk_workspace_bytes(...)              */
  REGTOPK_ERR_SEQUENCE = -3,            /* worker_step twice without aggregate, or aggregate first     */
  REGTOPK_ERR_CUDA = -4,                /* a CUDA runtime call or launch failed                        */
  REGTOPK_ERR_INTERNAL = -5,            /* the device reported an inconsistent selection (a bug)       */
  REGTOPK_ERR_NO_DEVICE = -6,           /* no usable sm_100 device / kernel image                      */
  REGTOPK_ERR_TOO_LARGE = -7            /* the problem exceeds a fixed built-in capacity               */
};

enum { REGTOPK_GRAD_F32 = 0, REGTOPK_GRAD_BF16 = 1 };

/* flags of regtopk_params */
enum {
  REGTOPK_FLAG_HOST_STAGING = 1,      /* reserve workspace for regtopk_round_host                          */
  REGTOPK_FLAG_FORCE_DENSE_SELECT = 2, /* testing: skip the sampled cutoff, always take the dense exact path */
  REGTOPK_FLAG_FORCE_WIDE_LISTS = 4,   /* testing: handle the candidate lists the way large N*k is handled (separate
                                          full-grid kernels, pairs unzipped afterwards) at any size; same results */
  REGTOPK_FLAG_GRID_DENSE_SELECT = 8,  /* testing: when a worker needs the dense exact path, run it as the full-grid
                                          kernel that large problems use, at any size; same results              */
  REGTOPK_FLAG_NUMERATORS_AT_AGGREGATE = 16 /* testing: form the numerators of the next round's distortion during the
                                          aggregation, as is done for large d, at any size; same results          */
};

typedef struct {
  float mu;            /* > 0: RegTop-k (Algorithm 2).  == 0: Top-k with error accumulation (Algorithm 1). */
  const float* omega;  /* host array of N aggregation weights (Eq. (1)), or NULL for 1/N each.             */
  int32_t grad_dtype;  /* REGTOPK_GRAD_F32 or REGTOPK_GRAD_BF16; accumulators and residuals are binary32.  */
  int32_t flags;       /* REGTOPK_FLAG_*                                                                   */
  float y;             /* exponent of Remark 3: selection metric |a|^y * regulariser, 0 < y <= 1; 0 or 1 means
                          Algorithm 2 as printed.  The mask is computed by ranking |a| * regulariser^(1/y), which
                          orders the entries the same way.                                                   */
  /* Layer-wise sparsification (one Top-k per layer instead of one over the whole vector; the paper's
     related-work section cites it).  n_layers == 0: Algorithm 2 as printed, one selection over all d
     coordinates.  n_layers >= 1: layer l is the contiguous index range [layer_end[l-1], layer_end[l])
     (layer_end ascending, layer_end[n_layers-1] == d) and keeps its layer_k[l] largest scores
     (1 <= layer_k[l] <= the layer's size); the k given to regtopk_create must equal the sum of layer_k.
     Accumulator, distortion, regulariser, sent values, residual and aggregation are unchanged; a worker's
     k pairs still come out in ascending index order.  Both arrays are host memory, read during
     regtopk_workspace_bytes and regtopk_create only.                                                     */
  int32_t n_layers;
  const int64_t* layer_end;
  const int64_t* layer_k;
} regtopk_params;

/* Bytes of device workspace a context for (d, N, k) needs; 0 if the arguments are invalid.
 * d = model size J, N = number of workers, k = entries kept per worker; 1 <= k <= d <= 2^31 - 2. */
size_t regtopk_workspace_bytes(int64_t d, int32_t N, int64_t k, const regtopk_params* params);

/* Algorithm 2, "Initialization": eps_n = 0 for every worker, no previous mask, round 0.
 * workspace: device memory, 256-byte aligned, at least regtopk_workspace_bytes(...) bytes; the library
 * keeps all state in it (residuals [N][ld] binary32, previous aggregate g [d], previous pairs, masks,
 * candidate lists).  cuda_stream: a cudaStream_t (NULL = default stream).  *out receives the context
 * (host).  Enqueues the clearing of the workspace.  Errors: INVALID_ARG, WORKSPACE_TOO_SMALL, CUDA,
 * NO_DEVICE. */
int regtopk_create(regtopk_ctx** out, int64_t d, int32_t N, int64_t k, const regtopk_params* params,
                   void* workspace, size_t workspace_bytes, void* cuda_stream);

/* One sparsification round of all N workers: Algorithm 2 steps 6-12 (Algorithm 1 steps 2-7 in round 0
 * or when mu == 0).
 *   grads    [N][grad_ld] gradients g_n^t in the context's grad_dtype, row n at grads + n*grad_ld
 *            elements; read-only.  grad_ld >= d.  Rows that are 16-byte aligned (an aligned base and
 *            grad_ld % 4 == 0 for fp32, grad_ld % 8 == 0 for bf16) take the vectorised path; any other
 *            layout is accepted and read element by element.
 *   out_idx  [N][k] int32: worker n's mask support in ascending order.
 *   out_val  [N][k] binary32: the accumulator a_n^t at those indices (not the score).
 * Exactly k pairs per worker are written.  Afterwards the residual state holds eps^{t+1}.
 * Errors: INVALID_ARG (NULL pointer, grad_ld < d), SEQUENCE (previous round not aggregated), CUDA. */
int regtopk_worker_step(regtopk_ctx* ctx, const void* grads, int64_t grad_ld, int32_t* out_idx,
                        float* out_val);

/* Accumulate-in-place form of the same round, for callers whose gradient computation can add into a
 * buffer (a backward pass that accumulates): Algorithm 2 step 7, a_n^t = eps_n^t + g_n^t, is then the
 * caller's own addition, and the library never reads a separate gradient array nor rewrites the
 * accumulator: 4 bytes of memory traffic per coordinate and worker instead of 12.
 *   regtopk_accumulator gives the device pointer to the library's rows ([N][*ld] binary32, row n at
 *   *dev_ptr + n * *ld, *ld >= d).  Between rounds row n holds eps_n^t.  Before
 *   regtopk_worker_step_inplace the caller, on the context's stream (or ordered before it), adds
 *   g_n^t[j] to element j of row n for j < d, in binary32 with a single round-to-nearest addition
 *   per element; elements [d, *ld) must stay 0.  The context's grad_dtype is not used by this form.
 *   regtopk_worker_step_inplace then does what regtopk_worker_step does after its accumulate step
 *   (steps 8-12), with the same outputs, errors and call order; the two forms may be mixed from round
 *   to round, and the results are bit-identical to regtopk_worker_step given the same gradients. */
int regtopk_accumulator(regtopk_ctx* ctx, float** dev_ptr, int64_t* ld);
int regtopk_worker_step_inplace(regtopk_ctx* ctx, int32_t* out_idx, float* out_val);

/* Server side of the round (Section 2.2): g^t = sum_n omega_n * ghat_n^t, workers added in the order
 * n = 0..N-1 with each product rounded before its addition, then the state roll for round t+1 (the
 * pairs just sent become the previous mask and a^{t} on it, g^t becomes g^{t-1}).
 *   out_g    [d] binary32 or NULL; if given, receives a copy of g^t.
 * Errors: SEQUENCE (no worker_step since the last aggregate), CUDA. */
int regtopk_aggregate(regtopk_ctx* ctx, float* out_g);

/* regtopk_aggregate fused with the model update of distributed SGD (Section 1: theta^{t+1} = theta^t -
 * eta^t g^t): after g^t is formed, theta[j] <- theta[j] - (eta * g^t[j]) (product rounded first) for every j
 * some worker sent; all other entries would change by eta * 0 and are left alone, which is the same
 * result bit for bit.  theta [d] binary32 (device), eta finite.  theta == NULL is regtopk_aggregate.
 * Errors as regtopk_aggregate, plus INVALID_ARG for a non-finite eta. */
int regtopk_aggregate_update(regtopk_ctx* ctx, float* theta, float eta, float* out_g);

/* Server side of the round when the N workers are spread over several GPUs (one process and one context per GPU,
 * each context holding a contiguous block of the workers; the paper's workers send their k pairs to a server,
 * Section 2.2, and here every GPU plays the server for itself).  After regtopk_worker_step each process all-gathers
 * the pairs of all workers (any transport; the data must be in this GPU's own memory, ordered by worker, before the
 * call) and calls this instead of regtopk_aggregate: g^t = sum over all n_total workers of omega_n * ghat_n^t,
 * added in the order n = 0..n_total-1 with each product rounded first, so that every GPU obtains the same g^t bit
 * for bit; then the state roll.  g^t is what the next round's distortion (Eq. (Delta_def)) is formed from, which is
 * why it must cover all workers and not only this context's.
 *   all_idx, all_val  [n_total][k] pairs of all workers (device), this context's own among them.
 *   omega_all         host array of n_total weights, or NULL for 1/n_total each.  The context itself must have been
 *                     created with its own workers' weights out of the same array (its default of 1/N would be
 *                     1/(workers of this context)).
 *   out_g             [d] or NULL.
 * Indices outside [0, d) are ignored.  Errors: INVALID_ARG, SEQUENCE (no worker_step since the last aggregate), CUDA. */
int regtopk_aggregate_gathered(regtopk_ctx* ctx, int32_t n_total, const int32_t* all_idx, const float* all_val,
                               const float* omega_all, float* out_g);

/* Device pointer to the library's own copy of the latest aggregate g^t ([d] binary32, inside the
 * workspace, valid until the next regtopk_aggregate is enqueued).  *dev_ptr is written on the host. */
int regtopk_global_gradient(regtopk_ctx* ctx, const float** dev_ptr);

/* Back to Algorithm 2's initial state: eps = 0, no previous mask, g = 0, round 0. */
int regtopk_state_reset(regtopk_ctx* ctx);

/* Checkpointing.  What Algorithm 2 carries from round to round (the residuals eps_n, the previous masks and the
 * accumulator values on them, the previous aggregate g^{t-1}, the round counter) can be copied out of the workspace
 * into a caller buffer of regtopk_state_bytes(ctx) bytes (device memory) and later copied into a context created
 * with the same d, N, k, mu, y and grad_dtype; the rounds that follow are then bit-identical to the ones the exporting
 * context would have run.  Export only between rounds (after regtopk_aggregate): otherwise SEQUENCE.
 * regtopk_state_export enqueues the copies on the context's stream; regtopk_state_import synchronises the stream
 * (it reads the blob's header) and returns INVALID_ARG if the blob does not belong to an identical problem,
 * WORKSPACE_TOO_SMALL if `bytes` is short. */
size_t regtopk_state_bytes(regtopk_ctx* ctx);
int regtopk_state_export(regtopk_ctx* ctx, void* dst, size_t bytes);
int regtopk_state_import(regtopk_ctx* ctx, const void* src, size_t bytes);

/* One whole round from HOST buffers: copies h_grads ([N][grad_ld], pinned memory recommended) to the
 * device staging area, runs regtopk_worker_step and regtopk_aggregate, copies the pairs (and g if
 * h_g != NULL) back to host memory, and SYNCHRONISES the stream before returning.  Needs
 * REGTOPK_FLAG_HOST_STAGING at creation and grad_ld <= d rounded up to a multiple of 1024 (the row
 * length reserved for staging).  h_idx [N][k], h_val [N][k], h_g [d] or NULL: host. */
int regtopk_round_host(regtopk_ctx* ctx, const void* h_grads, int64_t grad_ld, int32_t* h_idx,
                       float* h_val, float* h_g);

/* Synchronises the stream and returns REGTOPK_OK or the sticky error recorded by the device
 * (REGTOPK_ERR_INTERNAL) or by CUDA (REGTOPK_ERR_CUDA); a device error survives regtopk_state_reset.
 * REGTOPK_ERR_INTERNAL means that a consistency check of the selection failed (a bug in the library): the round in
 * which it happened may have left pairs, masks and residuals that do not belong together, so the state is to be
 * discarded (regtopk_state_reset, or import of an earlier export); the code stays set so that it cannot go unnoticed.
 * The checked build of the library (-DREGTOPK_DEBUG=1) also returns REGTOPK_ERR_INVALID_ARG here once an
 * accumulator was infinite or NaN (gradients must be finite), until the next regtopk_state_reset. */
int regtopk_status(regtopk_ctx* ctx);

typedef struct {
  int64_t rounds;               /* worker_step calls so far                                               */
  int64_t kernel_launches;      /* kernels launched by this context so far                                */
  int64_t dense_select_workers; /* worker-rounds that needed the dense exact path (sampled cutoff missed) */
  int64_t candidates_last;      /* candidates gathered in the last round, summed over workers             */
  int64_t candidate_capacity;   /* per-worker capacity of the candidate list                              */
  int64_t device_error_bits;    /* 0, or which internal consistency check failed (1 count, 2 dense, 4 refine; 8: a
                                   range check of the checked build, -DREGTOPK_DEBUG=1) */
  int64_t post_cluster_blocks;  /* thread blocks per worker in the selection kernel's clusters */
} regtopk_stats;

/* Synchronises the stream and fills *out (host). */
int regtopk_get_stats(regtopk_ctx* ctx, regtopk_stats* out);

/* Per-kernel timing with CUDA events on the context's stream.  enable != 0 starts recording an event
 * pair around the streaming accumulate kernel of every following worker_step (up to 4096 calls);
 * regtopk_profile_read synchronises and returns the summed milliseconds and the number of calls, then
 * clears the record.  Both outputs are host pointers. */
int regtopk_profile_enable(regtopk_ctx* ctx, int enable);
int regtopk_profile_read(regtopk_ctx* ctx, double* stream_kernel_ms, int64_t* calls);

/* Test introspection: device pointer to the residuals eps ([N][*ld] binary32, *ld >= d). */
int regtopk_debug_residual(regtopk_ctx* ctx, const float** dev_ptr, int64_t* ld);

/* Server aggregation from explicit pairs, for callers that cannot give the library any device memory of
 * their own to work in and cannot allocate at this point either: code running inside a memory-pool or
 * allocator callback, under a framework that has claimed the whole device, or in a process whose
 * policy forbids cudaMalloc after start-up.  (The paper has no counterpart; this is a convenience of
 * this library.)  It computes exactly what regtopk_aggregate computes, g = sum_n omega_n * ghat_n with
 * the workers added in the order 0..N-1, but takes the pairs as arguments and keeps its scratch (one
 * bitmask row per worker) in a fixed array that is part of the library image instead of a workspace.
 *   idx, val  [N][k] pairs as regtopk_worker_step writes them: per worker distinct indices in
 *             ascending order.  The pairs are the caller's data and are not trusted: a pair whose index
 *             lies outside [0, d) is ignored, and nothing outside the scratch rows and out_g is written
 *             whatever the arrays hold (rows that are not ascending or repeat an index give an
 *             unspecified but in-bounds result).  omega: HOST array of N weights, or NULL for 1/N each.
 *   out_g     [d] binary32, fully overwritten.
 * Limits: N <= REGTOPK_STATIC_MAX_WORKERS and N * ceil(d/32 rounded up to 4) <= REGTOPK_STATIC_SCRATCH_WORDS
 * (8 MiB of scratch, which every GPU that loads the library holds until the process exits); larger
 * problems return REGTOPK_ERR_TOO_LARGE and must use a context.  No cudaMalloc, cudaFree or other
 * allocating call is made.  The first call on each device looks up the scratch array's device address
 * (that device must be current) and should therefore come before any stream capture.  All calls on a
 * device share the one array and clear the part they use first: two calls whose work overlaps on the
 * GPU (different streams, or different threads) race; issue them on one stream or synchronise between
 * them.  Work is enqueued on cuda_stream; the call does not synchronise.
 * Errors: INVALID_ARG, TOO_LARGE, NO_DEVICE, CUDA. */
#define REGTOPK_STATIC_SCRATCH_WORDS (1u << 21)
#define REGTOPK_STATIC_MAX_WORKERS 64
int regtopk_aggregate_pairs_static(int64_t d, int32_t N, int64_t k, const int32_t* idx, const float* val,
                                   const float* omega, float* out_g, void* cuda_stream);

/* Frees the host-side context.  Synchronises the stream first.  The workspace is the caller's. */
int regtopk_destroy(regtopk_ctx* ctx);

/* Static, human-readable text for a return code. */
const char* regtopk_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* REGTOPK_H_ */
