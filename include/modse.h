/*
 * modse.h - C ABI of the MoDSE (Mixture of Diverse Size Experts) feed-forward
 * layer for NVIDIA B200 (sm_100a).
 *
 * The layer is the one of "Mixture of Diverse Size Experts" (arXiv 2409.12210):
 *   gate     G(x) = Softmax(KeepTopK(H(x), k)),  H(x) = x . W_g      (Sec. 2, Eq. 2-3)
 *   output   y    = sum_i G_i(x) E_i(x)                               (Sec. 3.1, Eq. 4)
 * where expert E_i is a bias-free SwiGLU feed-forward block (the Llama-2 FFN
 * the paper's models are built on, Sec. 4.1) whose hidden width h_i differs
 * from expert to expert (Sec. 3.1).  Experts outside the top-k have gate
 * softmax(-inf) = 0 and are never evaluated; every token is served by exactly
 * k experts (no capacity limit, no dropped tokens).
 *
 * Notation: T tokens, d = d_model, N experts, k = top_k, h[e] = hidden width of
 * expert e, S = sum_e h[e], off[e] = sum_{e'<e} h[e'].
 *
 * All pointers named "device" are CUDA device pointers owned by the caller.
 * The library allocates no device memory; every call only enqueues kernels on
 * the given stream and returns without synchronising.  No exception crosses
 * this boundary and no call aborts: errors are returned as modse_status_t.
 */
#ifndef MODSE_H
#define MODSE_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct modse_layer modse_layer_t; /* opaque host object owned by the library */

typedef enum {
    MODSE_OK = 0,
    MODSE_ERR_INVALID_ARG = 1,         /* NULL/misaligned pointer, size out of range            */
    MODSE_ERR_UNSUPPORTED = 2,         /* legal layer the CUDA path cannot run (see modse_create) */
    MODSE_ERR_WORKSPACE_TOO_SMALL = 3, /* workspace_bytes < modse_workspace_bytes(...)           */
    MODSE_ERR_STATE = 4,               /* backward without a matching saved forward              */
    MODSE_ERR_CUDA = 5,                /* a CUDA runtime/driver call or launch failed            */
    MODSE_ERR_DEVICE_TIMEOUT = 6,      /* a bounded wait inside a kernel expired                 */
    MODSE_ERR_DEVICE_BOUNDS = 7        /* a kernel met an index outside its buffers              */
} modse_status_t;

typedef enum {
    MODSE_F32 = 0, /* fp32 storage, fp32 FMA arithmetic                                   */
    MODSE_BF16 = 1 /* bf16 storage, tensor-core products with fp32 accumulation           */
} modse_dtype_t;

/* ---- layer object ------------------------------------------------------- */

/* Describes a layer (Sec. 3.1): d_model, N experts with hidden widths
 * ffn_sizes[0..N) (copied), and k.  Host only; touches no GPU.
 * Requirements: d_model >= 8 and a multiple of 8; 1 <= n_experts <= 256;
 * 1 <= top_k <= n_experts; every width >= 16 and a multiple of 16.
 * top_k > 2 is a legal layer the CUDA path does not run (MODSE_ERR_UNSUPPORTED).
 * The bf16 type further needs d_model % 128 == 0 and every width % 64 == 0
 * (checked by forward/backward, MODSE_ERR_UNSUPPORTED).
 * The pair rule of Eq. 5-6 is not enforced (query it with modse_check_pairs).
 * Returns NULL on error; modse_last_create_error() says why.                 */
modse_layer_t *modse_create(int d_model, int n_experts, const int *ffn_sizes, int top_k);
modse_status_t modse_last_create_error(void); /* per calling thread */
modse_status_t modse_destroy(modse_layer_t *layer); /* NULL is accepted */

/* Sec. 3.1, Eq. 5-6: returns 1 iff n_experts is even and every adjacent pair
 * (2p, 2p+1) - the pairs that the expert-pair allocation of Sec. 3.2 places on
 * one GPU each - has the same width sum 2h; *pair_sum_out (may be NULL) gets it. */
int modse_check_pairs(const int *ffn_sizes, int n_experts, int *pair_sum_out);

const char *modse_status_string(modse_status_t status);

/* ---- tensors ------------------------------------------------------------ */

/* Weights, all row-major in the layer dtype, 16-byte aligned device pointers:
 *   w_router [N, d]   row i gives logit i of H(x) = x . W_g             (Eq. 2)
 *   w_gate   [S, d]   rows off[e] .. off[e]+h[e]-1 belong to expert e
 *   w_up     [S, d]   same
 *   w_down   [d, S]   columns off[e] .. off[e]+h[e]-1 belong to expert e
 * Expert e computes  E_e(x) = W_down_e (silu(W_gate_e x) * (W_up_e x)).      */
typedef struct {
    const void *w_router;
    const void *w_gate;
    const void *w_up;
    const void *w_down;
} modse_weights_t;

/* Weight gradients, same shapes and layouts; dw_router is always fp32, the
 * others are in the layer dtype.  Overwritten (not accumulated) by backward;
 * rows/columns of an expert that received no token are written as zeros.    */
typedef struct {
    void *dw_router;
    void *dw_gate;
    void *dw_up;
    void *dw_down;
} modse_wgrads_t;

/* ---- calls -------------------------------------------------------------- */

/* Bytes of device scratch a forward (and its backward, if save_for_backward)
 * needs for n_tokens tokens.  0 on bad arguments.  The buffer must be 256-byte
 * aligned and is owned by the caller; its content after forward holds the
 * routing tables and, if saved, the activations backward consumes.           */
size_t modse_workspace_bytes(const modse_layer_t *layer, modse_dtype_t dtype, int n_tokens,
                             int save_for_backward);

/* Eq. 2-4.  x [T, d] and y [T, d] device, layer dtype, row-major.
 * Steps, all on `cuda_stream` (a cudaStream_t, NULL = legacy default stream):
 * router logits + top-k + gates, per-expert counts/offsets and the stable
 * permutation (expert groups ascending, tokens ascending inside a group),
 * gather into expert groups, grouped up/gate projection with SwiGLU, grouped
 * down projection, gate-weighted sum back in token order (slot 0 then slot 1).
 * n_tokens == 0 is MODSE_OK and does nothing.                                */
modse_status_t modse_forward(modse_layer_t *layer, modse_dtype_t dtype, const modse_weights_t *weights,
                             const void *x, int n_tokens, void *y, void *workspace,
                             size_t workspace_bytes, int save_for_backward, void *cuda_stream);

/* Exact gradient of modse_forward with the top-k selection held fixed (the
 * selection is piecewise constant in x).  Needs the workspace of a preceding
 * modse_forward(..., save_for_backward=1) on the same layer object, dtype and
 * n_tokens (else MODSE_ERR_STATE) and the same x and weights.  dy [T, d] is
 * the upstream gradient, dx [T, d] the result (layer dtype).  Gate and router
 * gradients are computed and kept in fp32.  May be called repeatedly on one
 * saved forward.                                                             */
modse_status_t modse_backward(modse_layer_t *layer, modse_dtype_t dtype, const modse_weights_t *weights,
                              const void *x, const void *dy, int n_tokens, void *dx,
                              const modse_wgrads_t *wgrads, void *workspace, size_t workspace_bytes,
                              void *cuda_stream);

/* Device pointers to the routing tables inside `workspace`, valid after a
 * forward with the same layer/n_tokens until the workspace is reused.  Any
 * output pointer may be NULL.  (Per-slot counts are what the paper's Appendix A
 * tables list as "top0"/"top1".)
 *   topk_idx [T,k] int32 (slot 0 = largest logit; ties go to the lower index)
 *   topk_gate [T,k] fp32, counts [N], counts_slot [k,N], offsets [N+1],
 *   row_of [T,k] (row of assignment (t,j) in expert-grouped order),
 *   token_of [k*T] (inverse map)                                             */
modse_status_t modse_get_routing(const modse_layer_t *layer, const void *workspace, int n_tokens,
                                 const int **topk_idx, const float **topk_gate, const int **counts,
                                 const int **counts_slot, const int **offsets, const int **row_of,
                                 const int **token_of);

/* Device pointers to the fp32 gate gradients dg [T,k] and logit gradients of
 * the kept logits dz [T,k] written by modse_backward.                        */
modse_status_t modse_get_gate_grads(const modse_layer_t *layer, const void *workspace, int n_tokens,
                                    const float **dg, const float **dz);

/* Synchronises the stream and reads the status word kernels write when a
 * bounded wait expires (MODSE_ERR_DEVICE_TIMEOUT) or an index check fails
 * (MODSE_ERR_DEVICE_BOUNDS); MODSE_OK if none did.  The word is cleared by the
 * next modse_forward.  Index checks are always on: every kernel that follows a
 * row or token index read from the routing tables compares it with the table's
 * extent first and skips the access if it lies outside.
 *
 * modse_set_debug_checks(layer, 1) (or the environment variable MODSE_DEBUG=1
 * at modse_create) adds guard blocks: every region of the workspace is followed
 * by 256 spare bytes whose head modse_forward fills with a pattern and this
 * call compares; a kernel that wrote past its region turns up as
 * MODSE_ERR_DEVICE_BOUNDS.  (The blocks are part of modse_workspace_bytes in
 * either mode.)  No counterpart in the paper.                                */
modse_status_t modse_check_device_status(modse_layer_t *layer, const void *workspace, void *cuda_stream);
modse_status_t modse_set_debug_checks(modse_layer_t *layer, int on);

/* Number of kernel launches the last forward/backward call on this layer
 * enqueued (for launch accounting in benchmarks).                            */
int modse_last_launch_count(const modse_layer_t *layer);

/* Auxiliary load-balance loss of Sec. 3.2, Eq. 7-10 (the Switch-Transformer loss):
 *   L_a = alpha * N * sum_i f_i * P_i,
 * p(x) = softmax over all N router logits, f_i = fraction of tokens whose largest
 * probability is expert i (Eq. 8; equals the slot-0 count / T), P_i = mean of p_i
 * over the batch (Eq. 10).
 *
 * modse_aux_loss evaluates it for the batch of the last modse_forward on this layer
 * and workspace: loss (1 float), f [N] and P [N] are device pointers written on the
 * stream (f and P may be NULL).
 *
 * modse_set_aux_loss(alpha) makes the following modse_backward calls differentiate
 * the objective  sum(dy * y) + L_a : dx and dw_router receive, in addition,
 * dL_a/dz[t,m] = (alpha N / T) p_m (f_m - sum_i f_i p_i) for every expert m (f is
 * piecewise constant and is held fixed).  alpha = 0 (default) switches it off.
 * The fp32 dz returned by modse_get_gate_grads stays the layer-output part only. */
modse_status_t modse_aux_loss(modse_layer_t *layer, const void *workspace, int n_tokens, float alpha, float *loss,
                              float *f, float *P, void *cuda_stream);
modse_status_t modse_set_aux_loss(modse_layer_t *layer, float alpha);

/* Output precision of a bf16 layer.  Off (default): y, dx and the expert weight
 * gradients are bf16 like the inputs.  On: the same fp32 accumulators are
 * written as fp32 instead ([T,d] y and dx, [S,d]/[d,S] weight gradients of 4
 * bytes per element), which removes the last bf16 rounding - e.g. for gradient
 * accumulation over micro-batches in fp32.  No effect on fp32 layers.        */
modse_status_t modse_set_output_f32(modse_layer_t *layer, int on);

/* Choice of kernel shape per device (no counterpart in the paper: a property of this implementation).
 * Each grouped product of the bf16 layer exists with 128-row tiles, with 256-row tiles computed by one CTA and
 * with 256-row tiles computed by a pair of CTAs; which is fastest for the two forward products depends on how
 * fast the GPU at hand feeds shared memory from L2, which differs between otherwise identical boards.
 * modse_tune_forward runs the forward pass (arguments as modse_forward) a few times per candidate on the caller's own buffers, times it with CUDA events, and keeps the fastest plan in
 * the layer object for all later calls.  It allocates no device memory, SYNCHRONISES the stream, and leaves y
 * and the workspace as one modse_forward would.  Results do not depend on the plan (the K order of every sum
 * is the same).  fp32 layers have one kernel shape: the call returns MODSE_OK at once.
 * The plan it finds is the fastest for forward passes run on their own (serving); inside a training step the
 * stages share the GPU's power budget and the library default (CTA pairs for every product) has been the faster
 * choice on every board measured, so training code need not call it.
 * modse_get_tile_plan returns the plan: -1 for the library default, else a bit set with, for product k (0 up/gate,
 * 1 down, 2 down dgrad, 3 down wgrad, 4 up/gate dgrad, 5 up/gate wgrad), bit 8 + k set: 256-row tiles computed
 * by a pair of CTAs on neighbouring SMs; otherwise bit k set: 256-row tiles computed by one CTA, clear: 128-row
 * tiles.  modse_set_tile_plan installs one (e.g. a plan found earlier on the same device). */
modse_status_t modse_tune_forward(modse_layer_t *layer, modse_dtype_t dtype, const modse_weights_t *weights,
                                  const void *x, int n_tokens, void *y, void *workspace, size_t workspace_bytes,
                                  int save_for_backward, void *cuda_stream);
int modse_get_tile_plan(const modse_layer_t *layer);
modse_status_t modse_set_tile_plan(modse_layer_t *layer, int plan);

/* Fusions across the permutation (bf16 layers; Sec. 2 Eq. 1 and Sec. 3.1 Eq. 4 say "select the top-k experts
 * and combine their outputs" and fix no intermediate buffers).  `flags` is a sum of
 *   MODSE_FUSE_GATHER   the up/gate product gathers its rows from x through the permutation (TMA row gather)
 *                       instead of reading the grouped copy of x; a forward that saves nothing for backward
 *                       then skips the permute kernel altogether;
 *   MODSE_FUSE_DG_ROWDOT  the gate gradient dg[t,j] = <dY_t W_down_e, Hm_row> / g is accumulated inside the
 *                       down-dgrad epilogue (one partial per 128 columns, summed in column order), so
 *                       backward no longer reads the fp32 expert outputs o;
 *   MODSE_FUSE_SCATTER  with fp32 outputs (modse_set_output_f32) and top_k <= 2: the down product adds its
 *                       rows straight into y and the up/gate dgrad into dx (both zeroed first; two addends
 *                       into a zeroed element commute, so the result is the same bits in any order), the
 *                       buffers o and dxp and the combine pass disappear; implies MODSE_FUSE_DG_ROWDOT.
 * A flag that does not apply to a call (fp32 layer, bf16 outputs, top_k > 2) is ignored by that call.
 * A backward call follows the forward call it belongs to.  Results: GATHER and SCATTER give the same bits as
 * the unfused path; DG_ROWDOT sums dg in another order (same tolerance).  Default: none.              */
#define MODSE_FUSE_GATHER 1
#define MODSE_FUSE_DG_ROWDOT 2
#define MODSE_FUSE_SCATTER 4
modse_status_t modse_set_fusion(modse_layer_t *layer, int flags);
int modse_get_fusion(const modse_layer_t *layer);

/* Second term of the router logits (Sec. 2, Eq. 2 with the RMSNorm and Softplus
 * definitions that follow it):
 *   H(x)_i = (x W_g)_i + RMSNorm(Softplus((x W_n)_i)),
 *   RMSNorm(v)_i = gamma v_i / sqrt(mean_j v_j^2 + eps),
 * read as: W_n is a second [N,d] router matrix, the mean runs over the N expert
 * entries of a token, gamma is one learnable scalar.  The term is a function of
 * x alone (the paper draws no random number here), so it is simply part of the
 * logits that top-k, the gates, the auxiliary loss and the backward pass see.
 *
 * modse_set_noise_gate: w_noise is a DEVICE pointer to [N,d] in the layer's
 * dtype, 16-byte aligned, borrowed until it is replaced (it must stay valid for
 * every later forward/backward); NULL switches the term off (the default).
 * gamma any finite value, eps >= 0.
 * modse_set_noise_grads: where modse_backward writes dW_n ([N,d] fp32, device,
 * 16-byte aligned) and dgamma (one fp32, device); both overwritten.  Required
 * before a backward whose forward ran with the term on (else
 * MODSE_ERR_INVALID_ARG); a backward whose on/off state differs from its
 * forward's returns MODSE_ERR_STATE.
 * dx and the router gradients then include the term's contribution; every sum
 * has a fixed order as elsewhere.                                            */
modse_status_t modse_set_noise_gate(modse_layer_t *layer, const void *w_noise, float gamma, float eps);
modse_status_t modse_set_noise_grads(modse_layer_t *layer, float *dw_noise, float *dgamma);

/* Routing only, with no device allocation by anyone.  (The paper has no
 * counterpart: this is a packaging variant of the router stage of Eq. 2-3.)
 *
 * For callers that cannot allocate device memory - a plugin invoked from a
 * framework callback where cudaMalloc is off limits because it synchronises
 * the device and can fail mid-step, code living inside a memory pool it does
 * not own, or a tool that only wants the routing tables - the scratch of the
 * router and rank kernels lives in a fixed 4 MiB array inside the library
 * (every GPU that loads the library holds it until the process exits).  The
 * caller passes only inputs and outputs, all device pointers:
 *   x [T,d], w_router [N,d]  in `dtype`, 16-byte aligned
 *   topk_idx [T,k] int32, topk_gate [T,k] fp32, counts [N], counts_slot [k,N],
 *   offsets [N+1], row_of [T,k], token_of [k*T]  - same meaning and the same
 *   values as modse_get_routing after modse_forward.
 * Limits: the scratch must fit the array - about 4*k*T*3 + 1016*N bytes plus
 * k*N*4 bytes per 64 tokens, e.g. T <= 100000 tokens for 8 experts, top-2;
 * larger batches return MODSE_ERR_WORKSPACE_TOO_SMALL (nothing is launched).
 * modse_route_static_scratch_capacity() returns the array size in bytes.
 * The first call on each device looks up the array's device address (a host
 * call, no allocation); make that first call before any stream capture.
 * All calls share the one array and it keeps the last call's contents (the
 * call clears what must start at zero): two calls that overlap on the GPU -
 * different streams, or different host threads - race on it; serialise them.
 * Calls no cudaMalloc/cudaFree and no allocating library routine.
 * The array's device address is cached per process and per device context:
 * serialise the first calls of several host threads, and do not use the
 * library across a cudaDeviceReset.
 * modse_route_static_scratch_status synchronises `cuda_stream` and returns what
 * the kernels of the last call on the current device recorded in the array's
 * status word (MODSE_OK, MODSE_ERR_DEVICE_BOUNDS, MODSE_ERR_DEVICE_TIMEOUT);
 * it plays the part of modse_check_device_status, which needs a workspace.   */
modse_status_t modse_route_static_scratch(modse_dtype_t dtype, int d_model, int n_experts, int top_k,
                                          const void *x, const void *w_router, int n_tokens, int *topk_idx,
                                          float *topk_gate, int *counts, int *counts_slot, int *offsets,
                                          int *row_of, int *token_of, void *cuda_stream);
size_t modse_route_static_scratch_capacity(void);
modse_status_t modse_route_static_scratch_status(void *cuda_stream);

/* Per-stage device timing (profiling aid).  After modse_stage_timing_begin the
 * next max_calls forward/backward calls on this layer bracket each of their
 * stages with a pair of CUDA events on the call's stream (no work is skipped
 * or reordered).  modse_stage_timing_end waits for those events, writes
 * ms_out[call * MODSE_N_STAGES + stage] (milliseconds; -1 for a stage the call
 * did not run), the number of calls seen, and switches timing off again.
 * Stages 0-5 belong to forward (router, rank, permute, up/gate GEMM + SwiGLU,
 * down GEMM, combine), 6-11 to backward (dg + permute of dY, down dgrad +
 * SwiGLU backward, down wgrad, up/gate dgrad, up/gate wgrad, router backward). */
#define MODSE_N_STAGES 12
modse_status_t modse_stage_timing_begin(modse_layer_t *layer, int max_calls);
modse_status_t modse_stage_timing_end(modse_layer_t *layer, float *ms_out, int *calls_out);
const char *modse_stage_name(int stage);

/* Debugging aid, process-wide: when on, bf16 layers run their grouped GEMMs on
 * the fp32-FMA kernels of the fp32 type (with bf16 storage) instead of the
 * tensor-core kernels - slow, meant for cross-checking.  Such a forward must
 * be called with save_for_backward = 1.  Off by default.                    */
void modse_debug_use_fma_path(int on);

/* Tuning aid, process-wide: the tile plan (see modse_get_tile_plan) of layers that have none of their own.
 * The library's default (0x3F3A) puts every product on CTA pairs, and, where that kernel does not apply (the
 * row-gathering up/gate product), products 1, 3, 4 and 5 on one-CTA 256-row tiles.  Every choice gives
 * bit-identical results (the order in which each output element is summed does not depend on the tile shape). */
void modse_debug_set_default_tile_plan(int plan);

/* Tuning aid, process-wide: 1 (default) - the CTAs of a grouped product take tiles, longest K first, from a
 * counter in the workspace; 0 - the tiles are dealt to the CTAs round-robin.  Same results either way.   */
void modse_debug_set_dynamic_tiles(int on);

/* Tuning aid, process-wide: how many warps of a CTA run the epilogue of a grouped product.  Bit k of mask_128 /
 * mask_256 / mask_pair set: product k (numbered as in modse_get_tile_plan) runs sixteen epilogue warps when it
 * is on 128-row tiles / one-CTA 256-row tiles / CTA-pair tiles, clear: eight.  Default: sixteen for the up/gate
 * product and the down dgrad on one-CTA 256-row tiles (mask_256 = 5), eight elsewhere.  Same results either way,
 * except that the gate gradient of MODSE_FUSE_DG_ROWDOT is summed from twice as many partials (same tolerance). */
void modse_debug_set_epilogue_warps(int mask_128, int mask_256, int mask_pair);

/* Failure-path aids, process-wide.  Every wait inside a kernel gives up after a limit (default 2000 ms),
 * records MODSE_ERR_DEVICE_TIMEOUT in the status word, lets its copies in flight land, frees its tensor
 * memory and returns; modse_debug_set_wait_limit_ms changes the limit (1..60000).
 * modse_debug_skip_tile_loads(product, tile) makes the CTA that is handed tile `tile` of grouped product
 * `product` (0..5) issue no loads for it and stop producing, so that its consumers run into that limit with
 * nothing in flight; (-1, -1) switches it off.  For tests of the time-out path on tiny inputs.          */
void modse_debug_set_wait_limit_ms(int ms);
void modse_debug_skip_tile_loads(int product, int tile);

/* Test aid: byte offsets, inside a workspace of the given shape, of the padded row table prow_of [T,k] and of
 * the guard block behind topk_idx, and the number of padded rows (the extent row indices are checked against). */
modse_status_t modse_debug_workspace_offsets(const modse_layer_t *layer, modse_dtype_t dtype, int n_tokens,
                                             int save_for_backward, size_t *prow_of_offset, size_t *first_guard_offset,
                                             int *padded_rows);

#ifdef __cplusplus
}
#endif
#endif /* MODSE_H */
