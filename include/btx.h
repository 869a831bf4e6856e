/*
 * btx.h -- C ABI of the B200 (sm_100a) MoE feed-forward hot path of Branch-Train-MiX
 * (arXiv 2403.07816).
 *
 * General conventions
 *   - Every tensor argument is a DEVICE pointer to caller-owned, row-major, contiguous memory,
 *     16-byte aligned, unless its description says "host".  The library never allocates or
 *     frees device memory and keeps no pointer after a call returns.  What it does keep, per
 *     process: one helper stream per device (btx_moe_backward), the multiprocessor count per
 *     device, the address of one static scratch array per device (btx_lb_loss_noalloc), and the
 *     calling thread's stage-timing hook (btx_set_stage_events).
 *   - The current device must be the one the buffers and `stream` belong to.
 *   - `stream` is a cudaStream_t passed as void*.  Calls enqueue work on it and return without
 *     synchronising; arguments are validated on the host before anything is launched.
 *   - Element type of x, weights, y, dy, dx is given by btx_moe_desc.dtype (BTX_F32: float,
 *     BTX_BF16: bfloat16 with fp32 accumulation).  Logits, gates, probabilities, the loss and all
 *     weight gradients are fp32.  Index outputs are int32.
 *   - A `workspace` serves one call at a time (its first 256 bytes hold the device status word,
 *     a routing ticket and the tile counters of the call's kernels); calls that may overlap on the
 *     GPU, e.g. on different streams, need a workspace (and `saved` buffer) each.
 *   - Errors: a btx_status is returned; nothing is launched when it is not BTX_OK.  Device-side
 *     bounded waits that expire are recorded in the workspace and read with btx_device_status.
 *
 * Notation: T tokens, d = d_model, F = d_ff, E experts (at most 64), k selected experts per token
 * (k = E under BTX_ROUTE_SOFT), R = T*k assignments.
 */
#ifndef BTX_H_
#define BTX_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  BTX_OK = 0,
  BTX_ERR_INVALID_ARG = 1,   /* null required pointer, bad size, misaligned pointer          */
  BTX_ERR_UNSUPPORTED = 2,   /* valid request outside what the kernels cover                 */
  BTX_ERR_WORKSPACE = 3,     /* workspace / saved buffer smaller than btx_moe_sizes reports  */
  BTX_ERR_ARCH = 4,          /* current device is not compute capability 10.x                */
  BTX_ERR_CUDA = 5,          /* a CUDA runtime or driver call failed                         */
  BTX_ERR_TIMEOUT = 6        /* a device-side bounded wait expired (see btx_device_status)   */
} btx_status;

typedef enum { BTX_F32 = 0, BTX_BF16 = 1 } btx_dtype;

/* Routing function g (Section 3.2 and Section 3.3 "Routing method").
 *   TOPK   g = softmax over the k largest logits, zero elsewhere (the paper's default, k = 2).
 *   SWITCH k = 1; the gate is the full-softmax probability of the arg-max expert.
 *   SOFT   g = softmax over all E experts (every expert active); desc.k is ignored.
 *   SAMPLE1 "Sample Top-1": with the caller's Gumbel noise G[T,E] the soft sample is
 *          SoftMax((W_l x + G) / desc.gumbel_tau); only its largest entry is kept as the gate of that
 *          one expert (k = 1).  gumbel_tau = 0 is hard sampling, the paper's inference rule: expert
 *          arg-max(W_l x + G) with gate 1 and no router gradient.  Defined here without the
 *          load-balancing loss (lb_alpha must be 0); `probs` then holds the perturbed softmax.
 * Ties between equal logits go to the lower expert index; slot 0 holds the largest logit. */
typedef enum { BTX_ROUTE_TOPK = 0, BTX_ROUTE_SWITCH = 1, BTX_ROUTE_SOFT = 2, BTX_ROUTE_SAMPLE1 = 3 } btx_routing;

typedef struct {
  int32_t T, d_model, d_ff, E, k;
  int32_t dtype;              /* btx_dtype                                                     */
  int32_t routing;            /* btx_routing                                                   */
  float   lb_alpha;           /* alpha of the load-balancing loss (Section 3.3; 0.01 in 4.1.1) */
  int32_t lb_stopgrad_u;      /* 0: differentiate L_LB through u and p as printed; 1: u const  */
  int32_t save_for_backward;  /* forward fills `saved` so that btx_moe_backward can run        */
  int32_t skip_wgrad;         /* backward: experts frozen (the paper's freeze ablation, Section */
                              /* 4.3.1): no dW1/dW3/dW2, only dx and the router gradients       */
  float   gumbel_tau;         /* SAMPLE1 only: temperature of the Gumbel softmax; 0 = hard      */
  float   capacity_factor;    /* 0: no limit.  > 0 (Section 4.1 uses 1.5 for Switch routing): an */
                              /* expert accepts ceil(capacity_factor * T * k / E) assignments,   */
                              /* taken in order of t*k+slot; the rest are dropped: they add      */
                              /* nothing to y and receive no gradient through y.  Gates, probs,  */
                              /* u, p and the loss stay the router's.  Not valid with SOFT.      */
} btx_moe_desc;

/* Optional routing outputs of btx_moe_forward; any member may be NULL.  All device pointers.
 *   logits[T,E], probs[T,E] (full softmax), topk_idx[T,k], gates[T,k]; counts[E] tokens per
 *   expert, offsets[E+1] exclusive scan; perm[R]: sorted row -> t*k+slot with rows ordered by
 *   (expert ascending, token ascending); inv_perm[R] its inverse; u[E], p[E], lb_loss[1] of
 *   Section 3.3.  Under a capacity limit counts/offsets/perm cover the kept assignments only:
 *   perm reads -1 past offsets[E] and inv_perm reads -1 for a dropped assignment. */
typedef struct {
  float*   logits;
  int32_t* topk_idx;
  float*   gates;
  float*   probs;
  int32_t* counts;
  int32_t* offsets;
  int32_t* perm;
  int32_t* inv_perm;
  float*   u;
  float*   p;
  float*   lb_loss;
} btx_routing_out;

/* Bytes of `workspace` (scratch, contents undefined afterwards; one size serves forward and
 * backward) and of `saved` (forward -> backward state: routing, the expert-sorted copy of x and
 * the two SwiGLU pre-activations).  Host pointers out.  Sizes are upper bounds that do not depend
 * on the routing outcome. */
btx_status btx_moe_sizes(const btx_moe_desc* desc, size_t* workspace_bytes, size_t* saved_bytes);

/* FF_MoE(x) = sum_i g_i(W_l x) FF_i(x)  (Section 3.2), FF_i(x) = W2_i (silu(W1_i x) * W3_i x),
 * evaluated only for the selected experts, plus the load-balancing loss of Section 3.3.
 *   x[T,d]; w_router[E,d] (W_l); router_bias[E] fp32 or NULL (the paper has no bias);
 *   router_noise[T,E] fp32 Gumbel noise, required for BTX_ROUTE_SAMPLE1 and ignored otherwise;
 *   w1,w3[E,F,d]; w2[E,d,F]; y[T,d] out.  `routing` may be NULL.  `saved` may be NULL when
 *   desc.save_for_backward == 0.  d and F must be multiples of 8 in BF16 mode, of 4 in F32. */
btx_status btx_moe_forward(const btx_moe_desc* desc, const void* x, const void* w_router,
                           const float* router_bias, const float* router_noise,
                           const void* w1, const void* w3, const void* w2,
                           void* y, const btx_routing_out* routing, void* saved,
                           void* workspace, size_t workspace_bytes, void* stream);

/* Backward of btx_moe_forward for the scalar <y, dy> + lb_grad_scale * L_LB (MoE finetuning,
 * Sections 1 and 3.2; the loss is added to the training loss with weight 1, Section 3.3).
 * `saved` is the buffer the forward call filled with the same desc and inputs.
 * Outputs: dx[T,d] (dtype); dw_router[E,d], dbias[E] (may be NULL), dw1,dw3[E,F,d], dw2[E,d,F],
 * all fp32; dlogits[T,E] fp32 (may be NULL): the gradient with respect to the router logits W_l x that
 * dw_router, dbias and the router's share of dx are formed from (never accumulated into).
 * accumulate = 0 overwrites the weight gradients, 1 adds to them.  With desc.skip_wgrad
 * the three expert gradients are not computed and dw1, dw3, dw2 may be NULL.
 * The memory-bound router kernels run beside the weight-gradient GEMMs on a helper stream that the
 * library creates once per device (the only CUDA resource it keeps) and that is joined back into
 * `stream` before the call returns: everything is complete when `stream` is. */
btx_status btx_moe_backward(const btx_moe_desc* desc, const void* x, const void* w_router,
                            const float* router_bias, const float* router_noise,
                            const void* w1, const void* w3, const void* w2,
                            const void* dy, float lb_grad_scale, const void* saved,
                            void* dx, float* dw_router, float* dbias, float* dlogits,
                            float* dw1, float* dw3, float* dw2, int32_t accumulate,
                            void* workspace, size_t workspace_bytes, void* stream);

/* One training step of the layer with HOST activations: copies x_host, dy_host ([T,d], dtype;
 * pinned memory makes the copies asynchronous) into the device staging buffers x_dev, dy_dev,
 * runs btx_moe_forward (saving for backward) and btx_moe_backward, and copies y, dx and the
 * load-balancing loss back to y_host, dx_host, loss_host.  Weights, gradients, staging buffers,
 * `saved` and `workspace` are device memory as in the two calls it composes; desc.save_for_backward
 * must be 1.  Everything is ordered on `stream`; the host results are valid after the stream
 * has been synchronised.  `copy_stream` (optional, NULL = none) is a second stream of the caller on
 * which the dy upload overlaps the forward pass and the y download overlaps the backward pass; the
 * call joins it back into `stream` before it returns. */
btx_status btx_moe_step_host(const btx_moe_desc* desc, const void* x_host, const void* dy_host,
                             void* y_host, void* dx_host, float* loss_host,
                             void* x_dev, void* dy_dev, void* y_dev, void* dx_dev,
                             const void* w_router, const float* router_bias, const float* router_noise,
                             const void* w1, const void* w3, const void* w2, float lb_grad_scale,
                             float* dw_router, float* dbias, float* dw1, float* dw3, float* dw2,
                             int32_t accumulate, void* saved, void* workspace, size_t workspace_bytes,
                             void* stream, void* copy_stream);

/* L_LB = alpha * E * sum_i u_i p_i with u_i the batch mean of the gate of expert i and p_i the
 * batch mean of SoftMax_i (Section 3.3), from given fp32 logits[T,E]; router_bias[E] fp32 is added
 * to every row first (NULL: none, as in the paper).  Outputs loss[1], u[E], p[E]; dlogits[T,E]
 * (d loss / d logits) unless NULL.  Uses desc.T, E, k, routing (not SAMPLE1), lb_alpha,
 * lb_stopgrad_u.  Workspace: btx_lb_loss_workspace_size. */
btx_status btx_lb_loss_workspace_size(const btx_moe_desc* desc, size_t* workspace_bytes);
btx_status btx_lb_loss(const btx_moe_desc* desc, const float* logits, const float* router_bias, float* loss,
                       float* u, float* p, float* dlogits, void* workspace, size_t workspace_bytes, void* stream);

/* btx_lb_loss without a caller-supplied workspace (the paper has no counterpart; this is a
 * packaging variant of the call above).  It is meant for callers that hold no allocator: plug-in
 * code that is handed tensors by a host framework whose memory pool owns all device memory, or a
 * training loop that must not pay for the device-wide synchronisation a cudaMalloc implies.  The
 * scratch lives in a 4 MiB (BTX_LB_NOALLOC_SCRATCH_BYTES) static device array inside the library,
 * which every GPU that loads the library holds until the process exits.  Same arguments and
 * results as btx_lb_loss; inputs and outputs are still the caller's.
 *   - A request is refused with BTX_ERR_WORKSPACE, before anything is enqueued, exactly when
 *     btx_lb_loss_workspace_size(desc) exceeds the array (4 MiB covers e.g. T = 32768 tokens with
 *     E = 4, top-2, which needs 3.05 MiB).
 *   - The first call on each device looks up the array's device address (once per device, with that
 *     device current); make that first call before starting any stream capture.
 *   - The call allocates and frees nothing.  All calls on one device share the array, which keeps
 *     whatever the previous call left in it (the call itself clears the part that must start at
 *     zero): two calls whose kernels may overlap on the GPU, e.g. on different streams, race. */
#define BTX_LB_NOALLOC_SCRATCH_BYTES (4u << 20)
btx_status btx_lb_loss_noalloc(const btx_moe_desc* desc, const float* logits, const float* router_bias, float* loss,
                               float* u, float* p, float* dlogits, void* stream);

/* MiX merge (Section 3.2): the feed-forward matrices of the N expert LLMs become the experts of
 * one MoE layer (kind FFN: dst[e*numel .. ] = src[e], bit for bit); every other parameter is the
 * uniform mean over the N models (kind AVERAGE: fp32 sum in model order, divided by N, rounded
 * once to dtype).  `items` is a HOST array; each item's `src` is a HOST array of N device
 * pointers.  Sources and destinations must not overlap.  numel*sizeof(element) need not be a
 * multiple of 16 for AVERAGE items; the pointers must be 16-byte aligned.  The three FFN_W* kinds
 * name which matrix an item is and are all stacked like BTX_PARAM_FFN.
 * The item table is staged through pageable host memory inside the call: the call blocks the host
 * for that copy and must not be recorded into a CUDA graph. */
typedef enum { BTX_PARAM_AVERAGE = 0, BTX_PARAM_FFN = 1, BTX_PARAM_FFN_W1 = 1, BTX_PARAM_FFN_W3 = 2,
               BTX_PARAM_FFN_W2 = 3 } btx_param_kind;
typedef struct {
  int32_t kind;               /* btx_param_kind */
  int32_t layer;              /* informational  */
  uint64_t numel;             /* elements per source tensor */
  const void* const* src;     /* host array of n_models device pointers */
  void* dst;                  /* device; numel elements (AVERAGE) or n_models*numel (FFN) */
} btx_merge_item;

btx_status btx_merge_workspace_size(int32_t n_models, uint64_t n_items, size_t* workspace_bytes);
btx_status btx_merge(int32_t n_models, int32_t dtype, const btx_merge_item* items, uint64_t n_items,
                     void* workspace, size_t workspace_bytes, void* stream);

/* Feed-forward layouts of the MiX merge for ONE layer (Section 3.2 and Section 3.3 "Splitting Experts",
 * "Blending Experts").  Sources: per model i, W1_i, W3_i [F,d] and W2_i [d,F] (host arrays of N device
 * pointers).  Destinations: w1_dst, w3_dst [E',F',d], w2_dst [E',d,F'].
 *   STACK  E' = N, F' = F: expert i is model i's FFN (what BTX_PARAM_FFN items do).
 *   SPLIT  E' = N*chunks, F' = F/chunks: expert i*chunks+c holds hidden units c*F' .. (c+1)*F' of model i
 *          (rows of W1/W3, columns of W2), so the un-gated sum of the chunks of model i equals FF_i.
 *   BLEND  E' = N, F' = F (chunks is ignored, N chunks are used): expert n holds the n-th chunk of every
 *          model, model i's chunk in hidden units i*F/N .. (i+1)*F/N.
 * All copies are bit-exact.  F/chunks and d must span whole 16-byte vectors. */
typedef enum { BTX_FFN_STACK = 0, BTX_FFN_SPLIT = 1, BTX_FFN_BLEND = 2 } btx_ffn_layout;
btx_status btx_merge_ffn_workspace_size(int32_t n_models, int32_t chunks, size_t* workspace_bytes);
btx_status btx_merge_ffn(int32_t n_models, int32_t dtype, int32_t layout, int32_t chunks, int32_t d_model,
                         int32_t d_ff, const void* const* w1_src, const void* const* w3_src,
                         const void* const* w2_src, void* w1_dst, void* w3_dst, void* w2_dst,
                         void* workspace, size_t workspace_bytes, void* stream);

/* Synchronises `stream` and reads the status word that kernels of earlier calls left in
 * `workspace`: *device_status (host) is BTX_OK or BTX_ERR_TIMEOUT. */
btx_status btx_device_status(const void* workspace, void* stream, int32_t* device_status);

/* Self-test of the bounded device-side waits (the paper has no counterpart).  Clears the status block at
 * the start of `workspace` (at least 256 bytes) and runs a kernel in which one thread waits, with a 50 ms
 * limit, on a barrier nobody arrives at: the wait gives up, records BTX_ERR_TIMEOUT in the status word and
 * the kernel returns normally, which is what every wait of the tensor-core kernels does (after about two
 * seconds) if a copy or a partner CTA never signals.  btx_device_status then reports BTX_ERR_TIMEOUT; the
 * CUDA context stays usable and the next call that uses the workspace clears the word again. */
btx_status btx_selftest_wait_expiry(void* workspace, size_t workspace_bytes, void* stream);

/* Optional stage timing for the calling host thread.  `events` is a host array of n
 * cudaEvent_t (as void*), or NULL to switch the hook off.  While set, btx_moe_forward records
 * events[0..4] on its stream: start, after routing+permutation+gather, after GEMM-1 (W1/W3 +
 * SwiGLU), after GEMM-2 (W2 + gate scatter), after combine; btx_moe_backward records
 * events[0..7]: start, after the dy gather, after dgrad-2, after dgrad-1, after the W2, W1 and W3
 * weight gradients, after the router backward.  Entries beyond n, or NULL entries, are skipped. */
btx_status btx_set_stage_events(void* const* events, int32_t n);

const char* btx_status_string(btx_status s);
int32_t btx_version(void);

#ifdef __cplusplus
}
#endif
#endif /* BTX_H_ */
