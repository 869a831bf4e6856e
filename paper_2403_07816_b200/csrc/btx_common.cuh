// Shared declarations of the btx CUDA library: the internal buffer plan, kernel launchers
// and small device helpers.  Nothing here is part of the public ABI (see include/btx.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "btx.h"

namespace btx {

constexpr int kRowTile = 256;        // expert segments of the sorted buffers are padded to this many rows
constexpr int kMaxExperts = 64;
constexpr int kMaxRouteBlocks = 1184; // bound of the router kernel's grid (sizes its partial-sum buffer)
constexpr int kStatusWords = 64;     // first 256 bytes of every workspace: device status block
                                     // (word 0: error code; word 8: ticket of the one-launch routing;
constexpr int kTileCounterWord = 16; //  words 16..23: tile counters of a call's tensor-core launches)

// ---------------------------------------------------------------------------------------------
// Buffer plan.  All offsets are bytes from the start of `saved` / `workspace`.
// ---------------------------------------------------------------------------------------------
struct Plan {
  int T, d, F, E, k, R;              // k = effective number of selected experts
  int esize;                         // bytes per element of dtype
  int r_pad_max;                     // upper bound of the padded sorted row count (multiple of kRowTile)
  int mt_max;                        // r_pad_max / kRowTile
  int nt_dact;                       // column tiles of the dgrad-2 GEMM (row-dot partials)
  int route_blocks;                  // blocks of the router kernel (partial sums for u, p)
  int perm_blocks;                   // blocks of the permutation kernels
  int wr_chunks;                     // token chunks of the router-weight gradient
  int small;                         // BF16 batch with T*k <= 1024: weight-streaming forward kernels
  int dec_s1, dec_s2;                // their contraction splits (pass 1: W1/W3, pass 2: W2)
  int dense;                         // a handful of tokens, nothing kept for backward: every expert meets all tokens
  int dense_n;                       // MMA N of that path: T rounded up to a multiple of 16
  int capacity;                      // rows one expert accepts (R when there is no limit)
  int capped;                        // a capacity limit is set: assignments may be dropped
  // saved
  size_t s_topk, s_gates, s_probs, s_logits, s_u, s_p, s_up64, s_loss, s_counts, s_offsets, s_pad_offsets,
      s_tile_expert, s_rowmap, s_flat2row, s_perm, s_inv_perm, s_xs, s_h1, s_h3, saved_bytes;
  // workspace
  size_t w_status, w_route_part, w_perm_counts, w_perm_base, w_act, w_yp, w_dys, w_dh1, w_dh3, w_ga,
      w_dxp, w_dg_part, w_dz, w_dwr_part, w_part, w_saved_fallback, workspace_bytes;
};

// routing_only: plan for btx_lb_loss (no expert buffers)
btx_status make_plan(const btx_moe_desc* desc, Plan* plan, bool routing_only);

// Pointers into saved/workspace resolved for one call.
struct Buffers {
  int32_t* topk;      float* gates;   float* probs;   float* logits;
  float* u;           float* p;       float* loss;
  double* up64;       // the batch means u[E] then p[E] as computed (double), for the backward
  int32_t* counts;    int32_t* offsets;   int32_t* pad_offsets;   int32_t* tile_expert;
  int32_t* rowmap;    // padded sorted row -> flat assignment id (t*k+slot), -1 for padding rows
  int32_t* flat2row;  // flat assignment id -> padded sorted row (-1: dropped by the capacity limit)
  int32_t* perm;      int32_t* inv_perm;
  void* xs;  void* h1;  void* h3;
  int32_t* status;    float* route_part;  int32_t* perm_counts;  int32_t* perm_base;
  void* act;  float* yp;  void* dys;  void* dh1;  void* dh3;  void* ga;  float* dxp;
  float* dg_part;  float* dz;  float* dwr_part;
  float* part;        // split partial products of the small-batch forward
};

// Records stage event i of the calling thread's timing hook (no-op when the hook is off).
void mark_stage(int i, cudaStream_t st);

// Multiprocessor count of the current device (looked up once per device).
int sm_count();

// ---------------------------------------------------------------------------------------------
// Launchers (defined in the .cu files).
// ---------------------------------------------------------------------------------------------
// `routing` is the effective rule (Sample Top-1 arrives as SWITCH, or TOPK for hard sampling, on the
// logits perturbed by `noise` and scaled by `inv_tau`; noise == nullptr: no perturbation).
cudaError_t launch_router(const Plan& pl, int dtype, int routing, float alpha, const void* x, const void* w_router,
                          const float* bias, const float* given_logits, const float* noise, float inv_tau,
                          const Buffers& b, cudaStream_t st);
cudaError_t launch_permute(const Plan& pl, const Buffers& b, cudaStream_t st);
cudaError_t launch_wait_expiry_selftest(int32_t* status, cudaStream_t st);
// Router + loss + permutation in one single-block launch, for batches with T*k <= 1024.
bool route_permute_small_fits(const Plan& pl);
cudaError_t launch_route_permute_small(const Plan& pl, int dtype, int routing, float alpha, const void* x,
                                       const void* w_router, const float* bias, const float* noise, float inv_tau,
                                       const Buffers& b, cudaStream_t st);
cudaError_t launch_gather_rows(const Plan& pl, const void* src, void* dst_sorted, const Buffers& b, cudaStream_t st);
// y[t] = sum over slots and over `splits` partial copies ([split][R][d]) of the expert rows
cudaError_t launch_combine(const Plan& pl, int dtype, const float* rows, int splits, void* y, const Buffers& b,
                           cudaStream_t st);
cudaError_t launch_router_backward(const Plan& pl, int dtype, int routing, float alpha, float lb_scale,
                                   int stopgrad_u, int have_dg, const void* x, const void* w_router, const Buffers& b,
                                   void* dx, float* dw_router, float* dbias, float* dlogits_out, int accumulate,
                                   float dz_scale, int perturbed, cudaStream_t st);

// Expert GEMMs: SIMT fp32 kernels for BTX_F32, tcgen05 kernels for BTX_BF16.
cudaError_t launch_expert_forward_f32(const Plan& pl, const void* w1, const void* w3, const void* w2,
                                      const Buffers& b, int save, cudaStream_t st);
cudaError_t launch_expert_backward_f32(const Plan& pl, const void* w1, const void* w3, const void* w2,
                                       const Buffers& b, float* dw1, float* dw3, float* dw2, int accumulate,
                                       int skip_wgrad, cudaEvent_t after_dx, cudaStream_t st);
btx_status launch_expert_forward_bf16(const Plan& pl, const void* w1, const void* w3, const void* w2,
                                      const Buffers& b, int save, cudaStream_t st);
int pick_decode_splits(int base_tiles, int kb_total);
btx_status launch_expert_forward_small_bf16(const Plan& pl, const void* w1, const void* w3, const void* w2,
                                            const Buffers& b, int save, cudaStream_t st);
// Whole forward for at most 64 tokens when nothing is kept for backward, as one cooperative kernel: routing,
// act[e] = SwiGLU(x W1_e^T, x W3_e^T) for every expert and all tokens, the gate-scaled rows W2_e act[e][t] of the
// selected (token, expert) pairs, and their sum y.  Clears the status word itself.
bool dense_small_fits(const Plan& pl, int save_for_backward);
btx_status launch_forward_small_fused_bf16(const Plan& pl, int routing, float alpha, const void* x, const void* w_router,
                                           const float* bias, const float* noise, float inv_tau, const void* w1,
                                           const void* w3, const void* w2, void* y, const Buffers& b, cudaStream_t st);
btx_status launch_expert_backward_bf16(const Plan& pl, const void* w1, const void* w3, const void* w2,
                                       const Buffers& b, float* dw1, float* dw3, float* dw2, int accumulate,
                                       int skip_wgrad, cudaEvent_t after_dx, cudaStream_t st);

// ---------------------------------------------------------------------------------------------
// Device helpers
// ---------------------------------------------------------------------------------------------
// Programmatic dependent launch.  A kernel launched with launch_after_predecessor(..., early = true)
// may become resident while the kernel before it in the stream still runs; grid_dependency_wait()
// returns once that kernel has completed and its writes are visible (at once in a normal launch),
// and must come before the first access to anything the earlier kernels wrote or still read.
// allow_dependents() lets the next kernel of the stream be scheduled as soon as every CTA of this
// one has started, so that its launch latency and set-up overlap this kernel's run.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void allow_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_after_predecessor(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                            bool early, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = early ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ float sigmoid_f32(float v) { return 1.0f / (1.0f + expf(-v)); }

// a = silu(h1) * h3
__device__ __forceinline__ float swiglu_f32(float h1, float h3) { return h1 * sigmoid_f32(h1) * h3; }

// Given dact = dL/da: dh1 = dact*h3*s*(1+h1*(1-s)), dh3 = dact*h1*s
__device__ __forceinline__ void swiglu_bwd_f32(float h1, float h3, float dact, float& dh1, float& dh3) {
  float s = sigmoid_f32(h1);
  dh1 = dact * h3 * s * (1.0f + h1 * (1.0f - s));
  dh3 = dact * h1 * s;
}

}  // namespace btx
