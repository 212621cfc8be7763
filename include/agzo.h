/*
 * agzo.h -- C ABI of the B200 (sm_100a) implementation of the per-step hot path of AGZO,
 * Activation-Guided Zeroth-Order optimisation.
 *
 * For every linear layer l with weight W_l (d_out x d_in) and the input activations of
 * the current minibatch H_l (d_in x m, given here as X = H^T, one token per row):
 *   1. Algorithm 1 (SubspaceExtract): an orthonormal basis A_l (d_in x r) of a rank-r
 *      subspace of col(H_l) by K steps of block power iteration from a Gaussian test
 *      matrix.  Stored as V = A^T: r rows of length d_in.
 *   2. Eq. (agzo-perturb): Delta_l = R_l A_l^T with R_l (d_out x r) i.i.d. N(0,1),
 *      regenerated from a counter-based seed every time it is needed; the d_out x d_in
 *      matrix Delta_l is never stored.
 *   3. Algorithm 2: W <- W + mu*Delta in place, loss, (two-point mode: W <- W - 2mu*Delta,
 *      loss,) the projected-gradient scalar g, and the fused restore-and-update pass.
 *
 * Conventions shared by all calls
 *   - Every data pointer is a DEVICE pointer unless its name starts with "h_" or the text
 *     says "host".  Layer descriptor arrays are HOST arrays, read during the call only.
 *   - W is [d_out][ldw] row-major (the layout of a torch nn.Linear weight), bf16 or fp32.
 *     X is [m][ldx] row-major, bf16 or fp32.  V is [r][ldv] row-major fp32, ldv >= d_in.
 *   - The library allocates no device memory.  Scratch comes from the workspace handed to
 *     agzo_create; it must stay valid and must not be touched by the caller while a call
 *     that uses it is in flight.  The library keeps no other pointer past a call.
 *   - All work is enqueued on the caller's stream (a cudaStream_t passed as void*) and the
 *     calls return without waiting for it, except where stated.  Calls that share a context
 *     must be issued on one stream or be ordered by the caller (they share the workspace).
 *     Two pieces of state the library itself carries from call to call are made safe across a
 *     change of stream: the new stream waits for the last upload of the layer tables, and
 *     staged R operand images written on another stream are rewritten instead of reused.
 *   - Every function returns an agzo_status; nothing throws, traps or aborts.  Argument
 *     errors are detected on the host before anything is launched.  Conditions that only
 *     the device can see (a rank-deficient panel, a wait that ran out) are written to a
 *     status word in the workspace and reported by agzo_poll.
 *   - Random streams: Philox4x32-10 with key = the 64-bit step seed and counter
 *     (b_lo, b_hi, layer_id, tag); b = e >> 2 where e is the row-major index of the element
 *     inside the matrix being drawn, which takes output word e & 3 of that block.
 *     tag 0 = R_l (d_out x r), tag 1 = Omega (m x r), tag 2 = dense direction,
 *     tag 3 = Gaussian right factor (r x d_in) of the LOZO comparison.
 *     Normals are Box-Muller on the word pairs (x0,x1) and (x2,x3):
 *       u1 = ((x >> 8) + 1) * 2^-24, u2 = (x' >> 8) * 2^-24, s = sqrt(-2 ln u1),
 *       even lane = s*cos(2 pi u2), odd lane = s*sin(2 pi u2), in fp32.
 */
#ifndef AGZO_H_
#define AGZO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct agzo_ctx agzo_ctx;

typedef enum agzo_status {
  AGZO_OK = 0,
  AGZO_ERR_INVALID_ARG = 1,   /* null pointer, bad size, bad alignment, r out of range      */
  AGZO_ERR_UNSUPPORTED = 2,   /* a dtype / mode combination the library does not implement  */
  AGZO_ERR_CUDA = 3,          /* a CUDA runtime call failed; agzo_last_cuda_error has the code */
  AGZO_ERR_WORKSPACE = 4,     /* workspace missing, misaligned or too small for these layers */
  AGZO_ERR_STATE = 5,         /* call made on a destroyed / foreign context                 */
  AGZO_ERR_TIMEOUT = 6,       /* a bounded device-side wait ran out (reported by agzo_poll)  */
  AGZO_ERR_CALLBACK = 7,      /* the loss callback of agzo_step, or the all-reduce callback
                                 of a token-sharded extraction, returned non-zero            */
  AGZO_WARN_RANK_DEFICIENT = 100 /* some panel had a column that depends on the columns before
                                    it (R_kk <= 1e-4 of the column's own length); that column
                                    of V is zero (reported by agzo_poll)                    */
} agzo_status;

typedef enum agzo_dtype { AGZO_BF16 = 0, AGZO_F32 = 1 } agzo_dtype;

#define AGZO_MAX_RANK 64
#define AGZO_MAX_LAYERS 4096

/* One linear layer.  Plain data, no ownership.  Fields a call does not use may be NULL/0:
 * the in-place passes ignore X, ldx, x_dtype, m; extraction ignores W, W16.               */
typedef struct agzo_layer {
  void*       W;        /* [d_out][ldw], w_dtype; perturbed and updated in place           */
  int64_t     ldw;      /* row pitch of W in elements, >= d_in                             */
  void*       W16;      /* optional bf16 compute copy of an fp32 master W, else NULL.  When
                           present, W is never perturbed: perturb writes
                           W16 = bf16(W + c*Delta), update writes W += c*Delta; W16 = bf16(W) */
  int64_t     ldw16;
  const void* X;        /* [m][ldx], x_dtype: H_l^T, read only by extraction               */
  int64_t     ldx;
  float*      V;        /* [r][ldv] fp32: A_l^T, written by extraction, read by the passes */
  int64_t     ldv;
  int32_t     w_dtype;  /* agzo_dtype of W                                                 */
  int32_t     x_dtype;  /* agzo_dtype of X                                                 */
  int32_t     d_out;
  int32_t     d_in;
  int32_t     m;        /* tokens (b*T of Section 3.1)                                     */
  int32_t     r;        /* 1 <= r <= min(AGZO_MAX_RANK, d_in, m)                           */
  uint32_t    layer_id; /* enters the Philox counter: the per-layer seed s_l of Algorithm 2 */
  uint32_t    reserved; /* must be 0                                                       */
} agzo_layer;

typedef struct agzo_params {
  uint64_t seed;  /* step seed (Philox key)                                                */
  float    eps;   /* smoothing parameter mu                                                */
  float    lr;    /* step size eta                                                         */
  int32_t  K;     /* power-iteration steps of Algorithm 1 (the paper uses 3), 0 <= K <= 16 */
  int32_t  mode;  /* 0: two-point g = (f+ - f-)/(2 mu); 1: Algorithm 2 as printed,
                     g = (f+ - f0)/mu                                                      */
} agzo_params;

/* Loss callback of agzo_step: run the model's forward on `stream` with the weights as they
 * are now and leave the scalar loss at d_loss (device, double: g is a difference of two
 * nearly equal losses, so an fp32 loss would cap its accuracy near 1e-3 relative).  phase: 0 = unperturbed
 * forward, during or after which the X buffers of the descriptors must have been filled
 * (Algorithm 2, step 1), 1 = at W + mu*Delta, 2 = at W - mu*Delta.  Return 0 on success. */
typedef int (*agzo_loss_fn)(void* user, void* stream, int phase, double* d_loss);

/* ---------------------------------------------------------------- context and workspace */

/* Bytes of workspace that every call on these layers needs (host only, no CUDA call).
 * A workspace sized for one layer list is also valid for any list whose per-field maxima
 * and layer count are not larger.  Error: INVALID_ARG for a bad descriptor.              */
agzo_status agzo_workspace_bytes(const agzo_layer* h_layers, int n, size_t* h_bytes);

/* Creates a context bound to CUDA device `device` that will use `workspace`
 * (device memory, 256-byte aligned, workspace_bytes long; owned by the caller, who frees
 * it after agzo_destroy).  Synchronous: it clears the device status word.                */
agzo_status agzo_create(agzo_ctx** out, int device, void* workspace, size_t workspace_bytes);
agzo_status agzo_destroy(agzo_ctx* ctx);

/* Options: "extract_path" 0 = automatic, 1 = CUDA-core fp32 kernels only, 2 = require the
 * tensor-core kernels (UNSUPPORTED at call time if a layer cannot use them), 3 = as 2 but
 * without the fused power-step kernel (T = X Q and Y = X^T T as two sweeps over X);
 * "rmw_path" selects the kernel of the in-place passes: 0 = automatic (bf16 weights with
 * 16-byte aligned rows and r >= "rmw_tc_min_rank", default 3, take the tensor-core kernel,
 * everything else the CUDA-core kernels), 1 = CUDA-core kernels only, 2 = tensor-core kernel
 * for every layer that allows it; tuning knobs of that kernel, 0 = chosen by rank:
 * "rmw_tc_slots" (shared-memory ring slots), "rmw_tc_inflight" (loads in flight per CTA),
 * "rmw_tc_panels" (column panels per work item, 1 or 2); "rmw_stage_r" 0 = when some layer's rank
 * exceeds 16 the split R operand of every 128-row tile is written once per pass to the scratch
 * area (d_out x 4 r' bytes per layer, r' = r rounded up to 16) and copied in by the pass instead of
 * being regenerated for every column panel (later passes with the same seed and layers, i.e. the
 * flip and the restore/update of the same step, find it there and skip the writing), 1 = never,
 * 2 = always;
 * "share_inputs" 1 (default) = consecutive layers whose X is the same buffer (same pointer, pitch,
 * m, d_in: q/k/v or gate/up of a transformer block) are served by one sweep over X per product,
 * with identical results; 0 = every layer sweeps its X itself;
 * "extract_fused" 1 = layers with r <= 16 and d_in <= 12288 on the tensor-core path run each
 * power step in the fused kernel in which X crosses HBM once (thread-block clusters of
 * ceil(d_in / 512) CTAs, or ceil(d_in / 768)), where that cluster size keeps at least 70 % of
 * the device's SMs busy; 2 = the same without the last condition (every cluster size
 * the device can launch) and also for layers that share their X with a neighbour (with 1 those
 * stay with the sweeps that serve the whole group) and for launch waves of at most 64 MiB of
 * activations (with 1 those take the sweeps too: their X is still in L2 at the next sweep);
 * 0 = off: two sweeps over X per power step.  Default 1;
 * "wave_bytes" = activation bytes grouped into one launch wave of extraction;
 * "extract_streams" 2 (default) = alternate waves use two scratch regions and two helper
 * streams forked from and joined to the caller's stream, so that one wave's short kernels
 * overlap the other's sweeps over X; 1 = waves strictly one after another;
 * "time_kernel_class" = one agzo_kernel_class whose launches get a CUDA event pair on the
 * caller's stream (0 = none), read back by agzo_read_counters;
 * "debug_fail_step_call" = n (test aid, 0 = off): the n-th internal call of agzo_step
 * (extract, perturb, [flip,] ghat, restore_update) returns AGZO_ERR_CUDA on the host before
 * launching anything, so that the step's error path can be exercised without a fault.    */
agzo_status agzo_set_option(agzo_ctx* ctx, const char* name, int64_t value);

/* Token-sharded extraction over data-parallel ranks.  Algorithm 1 touches the activations only
 * through the products H Omega = X^T Omega, H^T Q = X Q and H T = X^T T, and the tokens (the
 * columns of H, m = batch x sequence of them) enter the last one as a sum: with the batch split
 * over ranks, rank p holding the rows X_p of X from global token `token_offset` on,
 *     Y = X^T T = sum_p X_p^T (X_p Q),
 * so every rank computes its own term and the Y panels are summed over the ranks before each
 * qr(Y).  All ranks then hold the same Y, hence the same V, bit for bit.  The paper runs on one
 * device and has no counterpart of this call.
 *
 * fn: called on the host, K + 1 times per wave of layers, after the launches that produce the
 * wave's Y panels have been enqueued on `stream`.  `d_buf` is ONE contiguous device buffer of
 * `count` floats that holds all those panels (and alignment gaps, whose content is arbitrary);
 * fn must enqueue on `stream` an in-place sum of it over all ranks (an all-reduce, e.g.
 * ncclAllReduce(d_buf, d_buf, count, ncclFloat, ncclSum, comm, stream)) and return 0; a non-zero
 * return ends the call with AGZO_ERR_CALLBACK.  Every rank must pass the same layers (same
 * d_in, r, layer_id; m may differ), the same seed, K and options, so that the ranks make the
 * same sequence of calls with the same counts.
 * token_offset: global index of this rank's first token; row t of the local X is row
 * token_offset + t of the batch and draws that row of the Gaussian test matrix Omega.
 * fn = NULL (with token_offset 0) returns to single-rank extraction.  While fn is set, waves run
 * one after another on the caller's stream ("extract_streams" is taken as 1).
 * The buffer is owned by the library (it lies in the workspace); fn must not keep the pointer. */
typedef int (*agzo_allreduce_fn)(void* user, void* stream, float* d_buf, size_t count);
agzo_status agzo_set_allreduce(agzo_ctx* ctx, agzo_allreduce_fn fn, void* user, int64_t token_offset);

typedef enum agzo_kernel_class {
  AGZO_KC_NONE = 0,
  AGZO_KC_RMW = 1,        /* the in-place low-rank pass                                    */
  AGZO_KC_XT_T = 2,       /* Y = X^T T, CUDA-core kernel                                   */
  AGZO_KC_X_Q = 3,        /* T = X Q, CUDA-core kernel                                     */
  AGZO_KC_PANEL_QR = 4,   /* the three kernels of qr(Y) as one unit                        */
  AGZO_KC_TC_XT_T = 5,    /* Y = X^T T, tensor-core kernel                                 */
  AGZO_KC_TC_X_Q = 6,     /* T = X Q, tensor-core kernel                                   */
  AGZO_KC_OMEGA = 7,      /* Gaussian test matrix fill                                     */
  AGZO_KC_RMW_TC = 8,     /* the in-place low-rank pass, tensor-core kernel                */
  AGZO_KC_FUSED_POWER = 9 /* Y = X^T (X Q) in one pass over X, tensor-core cluster kernel  */
} agzo_kernel_class;

/* Measurement aid.  Waits for the timed launches recorded since the last read, then returns
 * their summed device time in milliseconds, how many there were, and the number of kernel
 * launches of every class the context has issued since the last read; all three counters
 * are reset.  Any output pointer may be NULL.  Synchronises with the timed events only.   */
agzo_status agzo_read_counters(agzo_ctx* ctx, double* h_ms, int64_t* h_timed_launches,
                               int64_t* h_total_launches);

/* Inspection aid.  Plans the layer array as agzo_extract_subspace would (the plan is kept for
 * the next call with the same array; its tables are uploaded on `stream`) and writes, per layer,
 * the thread-block cluster size with which its power steps run in the fused kernel, 0 for a
 * layer served by the two-sweep kernels (no X, the "extract_fused" / "extract_path" options,
 * its shape, an X shared with a neighbouring layer, or a launch wave small enough for L2).  h_cluster: host, n entries.  Launches
 * no kernel.                                                                               */
agzo_status agzo_query_fused(agzo_ctx* ctx, const agzo_layer* h_layers, int n, int32_t* h_cluster,
                             void* stream);

/* Inspection aid.  h_clusters[C], C = 1..16 (17 host entries, entry 0 is 0): how many thread-block
 * clusters of C CTAs of the fused power-step kernel the context's device holds at once (a cluster
 * lives inside one GPC, so the answer depends on the chip's GPC sizes); all 0 where the tensor-core
 * path is unavailable.  This is what "extract_fused" = 1 weighs when it picks a layer's cluster size. */
agzo_status agzo_query_cluster_capacity(agzo_ctx* ctx, int32_t* h_clusters);

/* Waits for the stream work of this context issued so far on `stream` and returns the
 * device status word: AGZO_OK, AGZO_WARN_RANK_DEFICIENT or AGZO_ERR_TIMEOUT; the word is
 * cleared.  The only synchronising call besides create.                                  */
agzo_status agzo_poll(agzo_ctx* ctx, void* stream);

const char* agzo_status_string(agzo_status s);
int         agzo_last_cuda_error(const agzo_ctx* ctx);

/* ---------------------------------------------------------------- Algorithm 1 */

/* SubspaceExtract(H_l, r_l, K) for every layer: Omega_l (m x r) Gaussian from
 * (seed, layer_id, tag 1); Y = H Omega; K times { Q = qr(Y); Y = H (H^T Q) }; A = qr(Y).Q.
 * qr is the unique thin factorisation with a positive diagonal.  Writes V = A^T.
 * X may be released as soon as the stream work of this call has completed.
 * Errors: INVALID_ARG (null X or V, r > min(d_in, m), ldv < d_in, K out of range),
 * WORKSPACE.  Rank-deficient panels are reported through agzo_poll.                      */
agzo_status agzo_extract_subspace(agzo_ctx* ctx, const agzo_layer* h_layers, int n,
                                  uint64_t seed, int K, void* stream);

/* ---------------------------------------------------------------- Eq. (agzo-perturb), Algorithm 2 */

/* W_l <- W_l + scale * R_l A_l^T for every layer, R_l regenerated from (seed, layer_id,
 * tag 0): step 2 of Algorithm 2 with scale = mu; the two-point flip is scale = -2 mu.
 * One fused read-modify-write pass; fp32 arithmetic, one rounding to the storage type.
 * With a W16 compute copy: W16 <- bf16(W + scale * Delta), W untouched.                   */
agzo_status agzo_perturb(agzo_ctx* ctx, const agzo_layer* h_layers, int n, uint64_t seed,
                         float scale, void* stream);

/* W_l <- W_l - scale * R_l A_l^T: the "restore" half of step 3 of Algorithm 2.  It is the
 * same pass as agzo_perturb with the opposite sign, not a bit-exact undo: in bf16 storage
 * mu*Delta can be below one ulp of W.  With a W16 copy: W16 <- bf16(W).                   */
agzo_status agzo_restore(agzo_ctx* ctx, const agzo_layer* h_layers, int n, uint64_t seed,
                         float scale, void* stream);

/* W_l <- W_l - lr * g * R_l A_l^T with g read from device memory (d_ghat): the "update"
 * half of step 3.  With a W16 copy the master is updated and W16 <- bf16(W).             */
agzo_status agzo_update(agzo_ctx* ctx, const agzo_layer* h_layers, int n, uint64_t seed,
                        float lr, const float* d_ghat, void* stream);

/* The projected-gradient scalar (Algorithm 2, step 3; Eq. agzo-estimator), on the device:
 * mode 0: *d_ghat = (*d_f_plus - *d_f_other) / (2 eps)   (f_other = f at W - eps*Delta)
 * mode 1: *d_ghat = (*d_f_plus - *d_f_other) / eps       (f_other = f0)
 * evaluated in double and rounded to fp32.                                               */
agzo_status agzo_ghat(agzo_ctx* ctx, const double* d_f_plus, const double* d_f_other,
                      float eps, int mode, float* d_ghat, void* stream);

/* Step 3 of Algorithm 2 as one pass: W_l <- W_l + c * R_l A_l^T with
 * mode 0: c = eps - lr*g (the weights sit at W - eps*Delta after the second forward),
 * mode 1: c = -(eps + lr*g) (the weights sit at W + eps*Delta), g read from d_ghat,
 * c formed in double and rounded to fp32.  With a W16 copy: W <- W - lr*g*Delta and
 * W16 <- bf16(W).                                                                        */
agzo_status agzo_restore_update(agzo_ctx* ctx, const agzo_layer* h_layers, int n,
                                uint64_t seed, float eps, float lr, int mode,
                                const float* d_ghat, void* stream);

/* One AGZO iteration (Algorithm 2): loss(phase 0) -> extract -> perturb(+eps) ->
 * loss(phase 1) -> [mode 0: perturb(-2 eps) -> loss(phase 2)] -> ghat -> restore_update.
 * d_losses2 (device, 2 doubles) receives f_plus and f_other (f_minus or f0), d_ghat (device,
 * 1 float) receives g.  Error behaviour: the step tracks where the weights sit
 * (W + c*Delta); if the callback fails (ERR_CALLBACK) or any of the library's own calls
 * after the first pass returns an error, the inverse pass of the outstanding c is enqueued
 * before the error is returned, so the weights are back at W (up to the rounding of one
 * pass).  A failure before the first pass leaves W untouched.                            */
agzo_status agzo_step(agzo_ctx* ctx, const agzo_layer* h_layers, int n,
                      const agzo_params* h_params, agzo_loss_fn loss, void* user,
                      double* d_losses2, float* d_ghat, void* stream);

/* Second case of Eq. (agzo-perturb), for parameters that are not matrices of a linear
 * layer: w <- w + scale * u with u ~ N(0, I) from (seed, layer_id, tag 2), n_elems
 * contiguous elements of `dtype`.  If d_scale is not NULL the coefficient is
 * scale * (*d_scale) (so that the update can use the device-side g).                     */
agzo_status agzo_perturb_dense(agzo_ctx* ctx, void* w, int64_t n_elems, int dtype,
                               uint64_t seed, uint32_t layer_id, float scale,
                               const float* d_scale, void* stream);

/* Data-independent right factor, for comparison runs with LOZO (Section 2, Eq. lozo-layer-perturb:
 * Delta_l = U_l V_l^T with both factors Gaussian): V_l (stored as r rows of length d_in) is filled
 * with i.i.d. N(0,1) from (seed, layer_id, tag 3), element e = k * d_in + d.  The in-place passes
 * then apply U_l V_l^T exactly as they apply R_l A_l^T; LOZO's 1 / r_l belongs in the caller's step
 * size.  Only V, ldv, r, d_in and layer_id of the descriptors are used.                    */
agzo_status agzo_fill_gaussian_basis(agzo_ctx* ctx, const agzo_layer* h_layers, int n, uint64_t seed,
                                     void* stream);

/* ---------------------------------------------------------------- allocation-free variant */

/* (No counterpart in the paper: this entry point exists for callers, not for the method.)
 * Algorithm 1 for ONE layer without a context or a workspace: the same kernels as
 * agzo_extract_subspace's CUDA-core path, with their scratch in a fixed 4 MiB array that is
 * part of the library image on every GPU that loads it.  It is meant for callers that cannot
 * allocate device memory where they need a subspace -- a forward hook that runs while
 * another framework owns (or has frozen) the allocator, a callback in which an allocation
 * would synchronise the device, a job whose memory is fixed up front.  X and V are still
 * the caller's.  The call itself performs no cudaMalloc / cudaFree and calls no library
 * routine that allocates.  (The very first call on a device makes the CUDA runtime load the
 * library's kernels, for which the driver may set device memory aside; from the second call
 * on a device the free device memory is the same before and after a call.)
 *   X [m][ldx] (x_dtype), V [r][ldv] fp32 out, d_rank_deficient: optional device int32 that
 *   receives 1 when a panel column was zeroed (see AGZO_WARN_RANK_DEFICIENT), else 0.
 * Limit: the scratch of the problem must fit the array,
 *   512 + 4 m r + 4 slabs r d_in + 4 r d_in + 8 ceil(d_in/128) r^2 + 8 r^2  <=  4 MiB
 *   (each term rounded up to 256 bytes; slabs = ceil(m / max(256, ceil32(ceil(m/32)))));
 *   for example m = 4096, d_in = 2048, r = 16 fits, m = 16384, d_in = 4096, r = 16 does not.
 *   Larger problems are refused with AGZO_ERR_WORKSPACE and nothing is launched.
 * Uses the CURRENT CUDA device.  The first call on each device looks up the array's device
 * address (cudaGetSymbolAddress); make that first call before starting any stream capture.
 * All calls on a device share the one array, which keeps the previous call's contents (the
 * call clears what must start clean).  Two calls whose GPU work can overlap -- different
 * streams without an ordering between them, or different host threads -- race on it: order
 * them on one stream or with events.  Other errors: INVALID_ARG, UNSUPPORTED, CUDA.        */
agzo_status agzo_extract_subspace_static(const void* X, int64_t ldx, int32_t x_dtype, int32_t m,
                                         int32_t d_in, int32_t r, int32_t K, uint64_t seed,
                                         uint32_t layer_id, float* V, int64_t ldv,
                                         int32_t* d_rank_deficient, void* stream);

/* ---------------------------------------------------------------- test exports */

/* Raw Philox words / normals of elements first .. first+n-1 of stream (seed, layer_id, tag)
 * written to device memory; used to check the generator bit for bit.                     */
agzo_status agzo_debug_philox(agzo_ctx* ctx, uint64_t seed, uint32_t layer_id, uint32_t tag,
                              uint64_t first, uint64_t n, uint32_t* d_words, void* stream);
agzo_status agzo_debug_gaussian(agzo_ctx* ctx, uint64_t seed, uint32_t layer_id, uint32_t tag,
                                uint64_t first, uint64_t n, float* d_vals, void* stream);

/* Test export, host only (no context, no device): the fused power step's work split.  Layer i has
 * h_tiles[i] token tiles; the tiles of the n layers form one list that is cut into
 * *h_shares = min(total, clusters) contiguous shares whose sizes differ by at most one tile.
 * Outputs, all host: h_tile0[i] the layer's first tile in the list, h_first[i] the first share
 * that meets the layer, h_parts[i] how many shares meet it (= its partial sums of Y after a power
 * step; 0 for a layer without tiles), h_share_begin[0 .. *h_shares] the first tile of every share
 * and the total (clusters + 1 entries of room).  AGZO_ERR_INVALID_ARG for clusters < 1, a negative
 * count or more than 2^30 tiles.                                                            */
agzo_status agzo_debug_fused_split(const int32_t* h_tiles, int n, int clusters, int32_t* h_tile0,
                                   int32_t* h_first, int32_t* h_parts, int32_t* h_share_begin,
                                   int32_t* h_shares);

/* Exercises the bounded device-side wait that every pipeline of the tensor-core kernels uses:
 * launches one small block that waits, with the library's own wait routine, on a barrier that
 * nothing ever completes.  The wait gives up after its time limit (two seconds), the block
 * records the condition in the status word and exits normally; the next agzo_poll returns
 * AGZO_ERR_TIMEOUT and the context stays usable.  UNSUPPORTED without the tensor-core path. */
agzo_status agzo_debug_wait_timeout(agzo_ctx* ctx, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* AGZO_H_ */
