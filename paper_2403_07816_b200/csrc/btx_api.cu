// C ABI entry points: argument validation, the buffer plan, and the launch sequences of the
// forward and backward passes (see include/btx.h for the contract of every call).
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>

#include "btx_common.cuh"

namespace btx {

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

btx_status make_plan(const btx_moe_desc* desc, Plan* pl, bool routing_only) {
  if (!desc || !pl) return BTX_ERR_INVALID_ARG;
  if (desc->T < 1 || desc->E < 1) return BTX_ERR_INVALID_ARG;
  if (!routing_only && (desc->d_model < 1 || desc->d_ff < 1)) return BTX_ERR_INVALID_ARG;
  if (desc->dtype != BTX_F32 && desc->dtype != BTX_BF16) return BTX_ERR_INVALID_ARG;
  if (desc->routing < BTX_ROUTE_TOPK || desc->routing > BTX_ROUTE_SAMPLE1) return BTX_ERR_INVALID_ARG;
  int k = desc->routing == BTX_ROUTE_SOFT ? desc->E : desc->k;
  if (k < 1 || k > desc->E) return BTX_ERR_INVALID_ARG;
  if ((desc->routing == BTX_ROUTE_SWITCH || desc->routing == BTX_ROUTE_SAMPLE1) && k != 1) return BTX_ERR_INVALID_ARG;
  if (desc->routing == BTX_ROUTE_SAMPLE1 && (desc->gumbel_tau < 0.f || desc->lb_alpha != 0.f)) return BTX_ERR_UNSUPPORTED;
  if (!(desc->capacity_factor >= 0.f)) return BTX_ERR_INVALID_ARG;
  if (desc->capacity_factor > 0.f && desc->routing == BTX_ROUTE_SOFT) return BTX_ERR_INVALID_ARG;
  if (desc->E > kMaxExperts) return BTX_ERR_UNSUPPORTED;
  const int gran = desc->dtype == BTX_BF16 ? 8 : 4;         // rows must be whole 16-byte vectors
  if (!routing_only && (desc->d_model % gran || desc->d_ff % gran)) return BTX_ERR_UNSUPPORTED;
  if ((long long)desc->T * k > (1ll << 28)) return BTX_ERR_UNSUPPORTED;

  Plan& p = *pl;
  memset(&p, 0, sizeof(p));
  p.T = desc->T; p.E = desc->E; p.k = k; p.R = p.T * k;
  p.d = routing_only ? 0 : desc->d_model;
  p.F = routing_only ? 0 : desc->d_ff;
  p.esize = desc->dtype == BTX_BF16 ? 2 : 4;
  p.capped = desc->capacity_factor > 0.f;
  p.capacity = p.R;
  if (p.capped) {     // ceil(CF * T * k / E) in double; never more than the R assignments there are
    const double c = ceil((double)desc->capacity_factor * (double)p.R / (double)p.E);
    if (c < (double)p.R) p.capacity = (int)c;
  }
  p.r_pad_max = (int)align_up((size_t)p.R + (size_t)p.E * (kRowTile - 1), kRowTile);
  p.mt_max = p.r_pad_max / kRowTile;
  p.nt_dact = desc->dtype == BTX_BF16 ? 2 * ((p.F + 255) / 256) : (p.F + 63) / 64;   // row-dot partials per row
  p.route_blocks = (p.T + 15) / 16;                       // a router block routes 16 (BF16) or 32 tokens at a time; the
  if (p.route_blocks > 4 * sm_count()) p.route_blocks = 4 * sm_count();   // blocks are persistent, up to four per multiprocessor
  if (p.route_blocks > kMaxRouteBlocks) p.route_blocks = kMaxRouteBlocks;
  p.perm_blocks = (p.R + 1023) / 1024;
  p.wr_chunks = (p.T + 127) / 128;
  // Small BF16 batches stream the expert weights through the swap-AB kernels (weights on the M side,
  // an expert's tokens on the N side); measured at the Llama-2-7B shape with E = 4 they beat the
  // training-shaped kernels up to the routing kernel's limit of 1024 assignments.
  p.small = !routing_only && desc->dtype == BTX_BF16 && route_permute_small_fits(p);
  if (p.small) {
    const int chunks = p.E < p.R ? p.E : p.R;             // typical: every expert holds one token chunk
    p.dec_s1 = pick_decode_splits(2 * chunks * ((p.F + 255) / 256), (p.d + 63) / 64);
    p.dec_s2 = pick_decode_splits(chunks * ((p.d + 255) / 256), (p.F + 63) / 64);
    p.dense = dense_small_fits(p, desc->save_for_backward) ? 1 : 0;
    p.dense_n = (p.T + 15) & ~15;
  }

  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
  const size_t rp = (size_t)p.r_pad_max;
  p.s_topk = take((size_t)p.R * 4);       p.s_gates = take((size_t)p.R * 4);
  p.s_probs = take((size_t)p.T * p.E * 4); p.s_logits = take((size_t)p.T * p.E * 4);
  p.s_u = take(p.E * 4);  p.s_p = take(p.E * 4);  p.s_up64 = take(2 * p.E * 8);  p.s_loss = take(4);
  p.s_counts = take(p.E * 4);  p.s_offsets = take((p.E + 1) * 4);  p.s_pad_offsets = take((p.E + 1) * 4);
  p.s_tile_expert = take((size_t)p.mt_max * 4);
  p.s_rowmap = take(rp * 4);  p.s_flat2row = take((size_t)p.R * 4);
  p.s_perm = take((size_t)p.R * 4);  p.s_inv_perm = take((size_t)p.R * 4);
  p.s_xs = take(rp * p.d * p.esize);
  p.s_h1 = take(rp * p.F * p.esize);
  p.s_h3 = take(rp * p.F * p.esize);
  p.saved_bytes = o;

  o = 0;
  p.w_status = take(kStatusWords * 4);
  p.w_route_part = take((size_t)p.route_blocks * 2 * p.E * 4);
  p.w_perm_counts = take((size_t)p.perm_blocks * p.E * 4);
  p.w_perm_base = take((size_t)p.perm_blocks * p.E * 4);
  p.w_dz = take((size_t)p.T * p.E * 4);
  p.w_dwr_part = take((size_t)p.wr_chunks * p.E * (p.d + 1) * 4);
  p.w_dg_part = take((size_t)p.nt_dact * rp * 4);
  // forward and backward scratch overlap: act | yp  vs  dys | dh1 | dh3 | ga | dxp
  size_t base = o;
  p.w_act = take(rp * p.F * p.esize);
  p.w_yp = take((size_t)p.R * p.d * 4);
  size_t fwd_end = o;
  o = base;
  p.w_dys = take(rp * p.d * p.esize);
  p.w_dh1 = take(rp * p.F * p.esize);
  p.w_dh3 = take(rp * p.F * p.esize);
  p.w_ga = take(rp * p.F * p.esize);
  p.w_dxp = take((size_t)p.R * p.d * 4);
  if (o < fwd_end) o = fwd_end;
  if (p.small) {
    const size_t n1 = (size_t)2 * p.dec_s1 * p.R * p.F, n2 = (size_t)p.dec_s2 * p.R * p.d;
    p.w_part = take((n1 > n2 ? n1 : n2) * 4);
  }
  // a forward that keeps nothing for backward parks its "saved" state here
  p.w_saved_fallback = take(p.saved_bytes);
  p.workspace_bytes = o;
  return BTX_OK;
}

static void resolve(const Plan& p, char* saved, char* ws, Buffers* b) {
  b->topk = (int32_t*)(saved + p.s_topk);   b->gates = (float*)(saved + p.s_gates);
  b->probs = (float*)(saved + p.s_probs);   b->logits = (float*)(saved + p.s_logits);
  b->u = (float*)(saved + p.s_u);  b->p = (float*)(saved + p.s_p);  b->loss = (float*)(saved + p.s_loss);
  b->up64 = (double*)(saved + p.s_up64);
  b->counts = (int32_t*)(saved + p.s_counts);  b->offsets = (int32_t*)(saved + p.s_offsets);
  b->pad_offsets = (int32_t*)(saved + p.s_pad_offsets);  b->tile_expert = (int32_t*)(saved + p.s_tile_expert);
  b->rowmap = (int32_t*)(saved + p.s_rowmap);  b->flat2row = (int32_t*)(saved + p.s_flat2row);
  b->perm = (int32_t*)(saved + p.s_perm);  b->inv_perm = (int32_t*)(saved + p.s_inv_perm);
  b->xs = saved + p.s_xs;  b->h1 = saved + p.s_h1;  b->h3 = saved + p.s_h3;
  b->status = (int32_t*)(ws + p.w_status);  b->route_part = (float*)(ws + p.w_route_part);
  b->perm_counts = (int32_t*)(ws + p.w_perm_counts);  b->perm_base = (int32_t*)(ws + p.w_perm_base);
  b->act = ws + p.w_act;  b->yp = (float*)(ws + p.w_yp);
  b->dys = ws + p.w_dys;  b->dh1 = ws + p.w_dh1;  b->dh3 = ws + p.w_dh3;  b->ga = ws + p.w_ga;
  b->dxp = (float*)(ws + p.w_dxp);
  b->part = (float*)(ws + p.w_part);
  b->dg_part = (float*)(ws + p.w_dg_part);  b->dz = (float*)(ws + p.w_dz);  b->dwr_part = (float*)(ws + p.w_dwr_part);
}

static thread_local void* const* g_stage_events = nullptr;
static thread_local int g_stage_count = 0;

void mark_stage(int i, cudaStream_t st) {
  if (g_stage_events != nullptr && i < g_stage_count && g_stage_events[i] != nullptr)
    cudaEventRecord((cudaEvent_t)g_stage_events[i], st);
}

// Sample Top-1 is Switch routing (soft sample) or top-1 with gate 1 (hard sample) on the logits
// perturbed by the Gumbel noise and divided by the temperature.
struct EffectiveRouting { int routing; float inv_tau; };
static EffectiveRouting effective_routing(const btx_moe_desc* desc) {
  if (desc->routing != BTX_ROUTE_SAMPLE1) return {desc->routing, 1.0f};
  if (desc->gumbel_tau > 0.f) return {BTX_ROUTE_SWITCH, 1.0f / desc->gumbel_tau};
  return {BTX_ROUTE_TOPK, 1.0f};
}

static bool misaligned(const void* p) { return ((uintptr_t)p & 15) != 0; }

// One helper stream per device, created on first use and kept for the life of the process: the
// backward pass runs its memory-bound router kernels on it beside the tensor-bound weight-gradient
// GEMMs.  nullptr when it cannot be had; the backward then runs on the caller's stream alone.
static cudaStream_t helper_stream() {
  static std::mutex mu;
  static cudaStream_t streams[64] = {};
  static bool failed[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(mu);
  if (streams[dev] == nullptr && !failed[dev]) {
    if (cudaStreamCreateWithFlags(&streams[dev], cudaStreamNonBlocking) != cudaSuccess) {
      streams[dev] = nullptr;
      failed[dev] = true;
      cudaGetLastError();
    }
  }
  return streams[dev];
}

struct ScopedEvents {                   // destroyed on every return path; destruction waits for nothing
  cudaEvent_t e[4] = {nullptr, nullptr, nullptr, nullptr};
  bool create(int n) {
    for (int i = 0; i < n; ++i)
      if (cudaEventCreateWithFlags(&e[i], cudaEventDisableTiming) != cudaSuccess) return false;
    return true;
  }
  ~ScopedEvents() { for (cudaEvent_t x : e) if (x) cudaEventDestroy(x); }
};

}  // namespace btx

int btx::sm_count() {
  constexpr int kMaxDevices = 64;
  static std::mutex mu;
  static int count[kMaxDevices] = {};
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    cudaGetLastError();
    return 148;                        // no usable device (size queries on a host without a GPU)
  }
  std::lock_guard<std::mutex> lock(mu);
  if (count[dev] == 0) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
      cudaGetLastError();
      return 148;
    }
    count[dev] = n;
  }
  return count[dev];
}

namespace btx {

static btx_status check_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return BTX_ERR_CUDA;
  int major = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return BTX_ERR_CUDA;
  return major == 10 ? BTX_OK : BTX_ERR_ARCH;
}

#define BTX_CUDA_OK(expr) do { if ((expr) != cudaSuccess) return BTX_ERR_CUDA; } while (0)

}  // namespace btx

using namespace btx;

extern "C" btx_status btx_moe_sizes(const btx_moe_desc* desc, size_t* workspace_bytes, size_t* saved_bytes) {
  Plan p;
  btx_status s = make_plan(desc, &p, false);
  if (s != BTX_OK) return s;
  if (workspace_bytes) *workspace_bytes = p.workspace_bytes;
  if (saved_bytes) *saved_bytes = p.saved_bytes;
  return BTX_OK;
}

extern "C" btx_status btx_moe_forward(const btx_moe_desc* desc, const void* x, const void* w_router,
                                      const float* router_bias, const float* router_noise, const void* w1,
                                      const void* w3, const void* w2,
                                      void* y, const btx_routing_out* routing, void* saved, void* workspace,
                                      size_t workspace_bytes, void* stream) {
  Plan pl;
  btx_status s = make_plan(desc, &pl, false);
  if (s != BTX_OK) return s;
  if (!x || !w_router || !w1 || !w3 || !w2 || !y || !workspace) return BTX_ERR_INVALID_ARG;
  if (desc->save_for_backward && !saved) return BTX_ERR_INVALID_ARG;
  if (desc->routing == BTX_ROUTE_SAMPLE1 && !router_noise) return BTX_ERR_INVALID_ARG;
  const EffectiveRouting er = effective_routing(desc);
  const float* noise = desc->routing == BTX_ROUTE_SAMPLE1 ? router_noise : nullptr;
  if (misaligned(x) || misaligned(w_router) || misaligned(w1) || misaligned(w3) || misaligned(w2) || misaligned(y) ||
      misaligned(workspace) || misaligned(saved))
    return BTX_ERR_INVALID_ARG;
  if (workspace_bytes < pl.workspace_bytes) return BTX_ERR_WORKSPACE;
  if ((s = check_device()) != BTX_OK) return s;

  cudaStream_t st = (cudaStream_t)stream;
  char* ws = (char*)workspace;
  char* sv = desc->save_for_backward ? (char*)saved : ws + pl.w_saved_fallback;
  Buffers b;
  resolve(pl, sv, ws, &b);

  mark_stage(0, st);
  // A handful of tokens, nothing kept: the whole layer is one cooperative kernel (it clears the status word
  // itself).  Where that launch is refused (a device partition with too few multiprocessors for all its
  // blocks to be resident at once, say) the launches below do the same work.
  bool done = false;
  if (pl.dense) {
    done = launch_forward_small_fused_bf16(pl, er.routing, desc->lb_alpha, x, w_router, router_bias, noise, er.inv_tau, w1,
                                           w3, w2, y, b, st) == BTX_OK;
    if (done) mark_stage(4, st);
    else cudaGetLastError();
  }
  if (!done) {
    const float* expert_rows = b.yp;
    int splits = 1;
    BTX_CUDA_OK(cudaMemsetAsync(b.status, 0, kStatusWords * 4, st));
    if (!route_permute_small_fits(pl) && pl.capacity < pl.R)       // the tail of perm past the kept rows reads -1
      BTX_CUDA_OK(cudaMemsetAsync(b.perm, 0xFF, (size_t)pl.R * sizeof(int32_t), st));
    if (route_permute_small_fits(pl)) {
      BTX_CUDA_OK(launch_route_permute_small(pl, desc->dtype, er.routing, desc->lb_alpha, x, w_router, router_bias, noise,
                                             er.inv_tau, b, st));
    } else {
      BTX_CUDA_OK(launch_router(pl, desc->dtype, er.routing, desc->lb_alpha, x, w_router, router_bias, nullptr, noise,
                                er.inv_tau, b, st));
      BTX_CUDA_OK(launch_permute(pl, b, st));
    }
    BTX_CUDA_OK(launch_gather_rows(pl, x, b.xs, b, st));
    mark_stage(1, st);
    if (desc->dtype == BTX_F32) {
      BTX_CUDA_OK(launch_expert_forward_f32(pl, w1, w3, w2, b, desc->save_for_backward, st));
    } else if (pl.small) {
      if ((s = launch_expert_forward_small_bf16(pl, w1, w3, w2, b, desc->save_for_backward, st)) != BTX_OK) return s;
      expert_rows = b.part;
      splits = pl.dec_s2;
    } else {
      if ((s = launch_expert_forward_bf16(pl, w1, w3, w2, b, desc->save_for_backward, st)) != BTX_OK) return s;
    }
    mark_stage(3, st);
    BTX_CUDA_OK(launch_combine(pl, desc->dtype, expert_rows, splits, y, b, st));
    mark_stage(4, st);
  }

  if (routing) {
    auto out = [&](void* dst, const void* src, size_t bytes) -> cudaError_t {
      return dst ? cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToDevice, st) : cudaSuccess;
    };
    BTX_CUDA_OK(out(routing->logits, b.logits, (size_t)pl.T * pl.E * 4));
    BTX_CUDA_OK(out(routing->probs, b.probs, (size_t)pl.T * pl.E * 4));
    BTX_CUDA_OK(out(routing->topk_idx, b.topk, (size_t)pl.R * 4));
    BTX_CUDA_OK(out(routing->gates, b.gates, (size_t)pl.R * 4));
    BTX_CUDA_OK(out(routing->counts, b.counts, pl.E * 4));
    BTX_CUDA_OK(out(routing->offsets, b.offsets, (pl.E + 1) * 4));
    BTX_CUDA_OK(out(routing->perm, b.perm, (size_t)pl.R * 4));
    BTX_CUDA_OK(out(routing->inv_perm, b.inv_perm, (size_t)pl.R * 4));
    BTX_CUDA_OK(out(routing->u, b.u, pl.E * 4));
    BTX_CUDA_OK(out(routing->p, b.p, pl.E * 4));
    BTX_CUDA_OK(out(routing->lb_loss, b.loss, 4));
  }
  return BTX_OK;
}

extern "C" btx_status btx_moe_backward(const btx_moe_desc* desc, const void* x, const void* w_router,
                                       const float* router_bias, const float* router_noise, const void* w1,
                                       const void* w3, const void* w2,
                                       const void* dy, float lb_grad_scale, const void* saved, void* dx,
                                       float* dw_router, float* dbias, float* dlogits, float* dw1, float* dw3,
                                       float* dw2, int32_t accumulate, void* workspace, size_t workspace_bytes,
                                       void* stream) {
  (void)router_bias;   // the bias only shifts the logits; its gradient needs dz alone
  (void)router_noise;  // likewise: the forward saved the perturbed probabilities
  Plan pl;
  btx_status s = make_plan(desc, &pl, false);
  if (s != BTX_OK) return s;
  const int skip_wgrad = desc->skip_wgrad != 0;
  if (!x || !w_router || !w1 || !w3 || !w2 || !dy || !saved || !dx || !dw_router || !workspace)
    return BTX_ERR_INVALID_ARG;
  if (!skip_wgrad && (!dw1 || !dw3 || !dw2)) return BTX_ERR_INVALID_ARG;
  if (misaligned(x) || misaligned(w_router) || misaligned(w1) || misaligned(w3) || misaligned(w2) ||
      misaligned(dy) || misaligned(saved) || misaligned(dx) || misaligned(dw_router) || misaligned(dlogits) ||
      misaligned(dw1) ||
      misaligned(dw3) || misaligned(dw2) || misaligned(workspace))
    return BTX_ERR_INVALID_ARG;
  if (workspace_bytes < pl.workspace_bytes) return BTX_ERR_WORKSPACE;
  if ((s = check_device()) != BTX_OK) return s;

  cudaStream_t st = (cudaStream_t)stream;
  Buffers b;
  resolve(pl, (char*)saved, (char*)workspace, &b);
  mark_stage(0, st);
  BTX_CUDA_OK(cudaMemsetAsync(b.status, 0, kStatusWords * 4, st));
  BTX_CUDA_OK(launch_gather_rows(pl, dy, b.dys, b, st));
  mark_stage(1, st);
  // The router backward (memory-bound, a few small kernels) depends on dgrad-2 and dgrad-1 only: it runs
  // on the helper stream beside the three tensor-bound weight-gradient GEMMs and joins `stream` at the end.
  ScopedEvents evs;
  cudaStream_t side = skip_wgrad ? nullptr : helper_stream();
  if (side != nullptr && !evs.create(2)) side = nullptr;
  cudaEvent_t after_dx = side != nullptr ? evs.e[0] : nullptr;
  if (desc->dtype == BTX_F32) {
    BTX_CUDA_OK(launch_expert_backward_f32(pl, w1, w3, w2, b, dw1, dw3, dw2, accumulate, skip_wgrad, after_dx, st));
  } else {
    if ((s = launch_expert_backward_bf16(pl, w1, w3, w2, b, dw1, dw3, dw2, accumulate, skip_wgrad, after_dx, st)) !=
        BTX_OK)
      return s;
  }
  const EffectiveRouting er = effective_routing(desc);
  cudaStream_t rst = side != nullptr ? side : st;
  if (side != nullptr) BTX_CUDA_OK(cudaStreamWaitEvent(side, after_dx, 0));
  BTX_CUDA_OK(launch_router_backward(pl, desc->dtype, er.routing, desc->lb_alpha, lb_grad_scale,
                                     desc->lb_stopgrad_u, 1, x, w_router, b, dx, dw_router, dbias, dlogits,
                                     accumulate, er.inv_tau, desc->routing == BTX_ROUTE_SAMPLE1, rst));
  if (side != nullptr) {
    BTX_CUDA_OK(cudaEventRecord(evs.e[1], side));
    BTX_CUDA_OK(cudaStreamWaitEvent(st, evs.e[1], 0));
  }
  mark_stage(7, st);
  return BTX_OK;
}

extern "C" btx_status btx_moe_step_host(const btx_moe_desc* desc, const void* x_host, const void* dy_host,
                                        void* y_host, void* dx_host, float* loss_host, void* x_dev, void* dy_dev,
                                        void* y_dev, void* dx_dev, const void* w_router, const float* router_bias,
                                        const float* router_noise, const void* w1, const void* w3, const void* w2, float lb_grad_scale,
                                        float* dw_router, float* dbias, float* dw1, float* dw3, float* dw2,
                                        int32_t accumulate, void* saved, void* workspace, size_t workspace_bytes,
                                        void* stream, void* copy_stream) {
  Plan pl;
  btx_status s = make_plan(desc, &pl, false);
  if (s != BTX_OK) return s;
  if (!x_host || !dy_host || !y_host || !dx_host || !loss_host || !x_dev || !dy_dev || !y_dev || !dx_dev || !saved)
    return BTX_ERR_INVALID_ARG;
  if (!desc->save_for_backward) return BTX_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  cudaStream_t cs = (cudaStream_t)copy_stream;
  const bool overlap = copy_stream != nullptr && copy_stream != stream;
  const size_t act_bytes = (size_t)pl.T * pl.d * pl.esize;
  ScopedEvents evs;
  cudaEvent_t &ev_start = evs.e[0], &ev_dy = evs.e[1], &ev_fwd = evs.e[2], &ev_y = evs.e[3];
  if (overlap) {
    // dy travels to the device while the forward runs, y travels back while the backward runs
    const unsigned f = cudaEventDisableTiming;
    if (cudaEventCreateWithFlags(&ev_start, f) != cudaSuccess || cudaEventCreateWithFlags(&ev_dy, f) != cudaSuccess ||
        cudaEventCreateWithFlags(&ev_fwd, f) != cudaSuccess || cudaEventCreateWithFlags(&ev_y, f) != cudaSuccess)
      return BTX_ERR_CUDA;
    BTX_CUDA_OK(cudaEventRecord(ev_start, st));             // the copy stream joins the caller's ordering
    BTX_CUDA_OK(cudaStreamWaitEvent(cs, ev_start, 0));
    BTX_CUDA_OK(cudaMemcpyAsync(dy_dev, dy_host, act_bytes, cudaMemcpyHostToDevice, cs));
    BTX_CUDA_OK(cudaEventRecord(ev_dy, cs));
  }
  BTX_CUDA_OK(cudaMemcpyAsync(x_dev, x_host, act_bytes, cudaMemcpyHostToDevice, st));
  if (!overlap) BTX_CUDA_OK(cudaMemcpyAsync(dy_dev, dy_host, act_bytes, cudaMemcpyHostToDevice, st));
  btx_routing_out ro;
  memset(&ro, 0, sizeof(ro));
  if ((s = btx_moe_forward(desc, x_dev, w_router, router_bias, router_noise, w1, w3, w2, y_dev, &ro, saved, workspace,
                           workspace_bytes, stream)) != BTX_OK)
    return s;
  if (overlap) {
    BTX_CUDA_OK(cudaEventRecord(ev_fwd, st));
    BTX_CUDA_OK(cudaStreamWaitEvent(cs, ev_fwd, 0));
    BTX_CUDA_OK(cudaMemcpyAsync(y_host, y_dev, act_bytes, cudaMemcpyDeviceToHost, cs));
    BTX_CUDA_OK(cudaEventRecord(ev_y, cs));
    BTX_CUDA_OK(cudaStreamWaitEvent(st, ev_dy, 0));
  }
  if ((s = btx_moe_backward(desc, x_dev, w_router, router_bias, router_noise, w1, w3, w2, dy_dev, lb_grad_scale, saved,
                            dx_dev, dw_router, dbias, nullptr, dw1, dw3, dw2, accumulate, workspace, workspace_bytes,
                            stream)) !=
      BTX_OK)
    return s;
  if (!overlap) BTX_CUDA_OK(cudaMemcpyAsync(y_host, y_dev, act_bytes, cudaMemcpyDeviceToHost, st));
  BTX_CUDA_OK(cudaMemcpyAsync(dx_host, dx_dev, act_bytes, cudaMemcpyDeviceToHost, st));
  BTX_CUDA_OK(cudaMemcpyAsync(loss_host, (const char*)saved + pl.s_loss, 4, cudaMemcpyDeviceToHost, st));
  if (overlap) {
    BTX_CUDA_OK(cudaStreamWaitEvent(st, ev_y, 0));          // everything is complete when `stream` is
  }
  return BTX_OK;
}

extern "C" btx_status btx_set_stage_events(void* const* events, int32_t n) {
  if (events != nullptr && n < 1) return BTX_ERR_INVALID_ARG;
  g_stage_events = events;
  g_stage_count = events ? n : 0;
  return BTX_OK;
}

extern "C" btx_status btx_lb_loss_workspace_size(const btx_moe_desc* desc, size_t* workspace_bytes) {
  Plan p;
  btx_status s = make_plan(desc, &p, true);
  if (s != BTX_OK) return s;
  if (!workspace_bytes) return BTX_ERR_INVALID_ARG;
  *workspace_bytes = p.workspace_bytes;
  return BTX_OK;
}

// Host-side checks shared by the two loss entry points (everything except the workspace).
static btx_status lb_loss_validate(const btx_moe_desc* desc, const float* logits, float* loss, float* u, float* p,
                                   Plan* pl) {
  btx_status s = make_plan(desc, pl, true);
  if (s != BTX_OK) return s;
  if (desc->routing == BTX_ROUTE_SAMPLE1) return BTX_ERR_UNSUPPORTED;
  if (!logits || !loss || !u || !p) return BTX_ERR_INVALID_ARG;
  return BTX_OK;
}

extern "C" btx_status btx_lb_loss(const btx_moe_desc* desc, const float* logits, const float* router_bias, float* loss,
                                  float* u, float* p, float* dlogits, void* workspace, size_t workspace_bytes,
                                  void* stream) {
  // every check comes before the first enqueue: a refused call leaves the stream and the workspace alone
  Plan pl;
  btx_status s = lb_loss_validate(desc, logits, loss, u, p, &pl);
  if (s != BTX_OK) return s;
  if (!workspace || misaligned(workspace)) return BTX_ERR_INVALID_ARG;
  if (workspace_bytes < pl.workspace_bytes) return BTX_ERR_WORKSPACE;
  if ((s = check_device()) != BTX_OK) return s;
  cudaStream_t st = (cudaStream_t)stream;
  char* ws = (char*)workspace;
  Buffers b;
  resolve(pl, ws + pl.w_saved_fallback, ws, &b);
  BTX_CUDA_OK(cudaMemsetAsync(b.status, 0, kStatusWords * 4, st));
  BTX_CUDA_OK(launch_router(pl, BTX_F32, desc->routing, desc->lb_alpha, nullptr, nullptr, router_bias, logits, nullptr,
                            1.0f, b, st));
  BTX_CUDA_OK(cudaMemcpyAsync(loss, b.loss, 4, cudaMemcpyDeviceToDevice, st));
  BTX_CUDA_OK(cudaMemcpyAsync(u, b.u, pl.E * 4, cudaMemcpyDeviceToDevice, st));
  BTX_CUDA_OK(cudaMemcpyAsync(p, b.p, pl.E * 4, cudaMemcpyDeviceToDevice, st));
  if (dlogits) {
    BTX_CUDA_OK(launch_router_backward(pl, BTX_F32, desc->routing, desc->lb_alpha, 1.0f, desc->lb_stopgrad_u, 0,
                                       nullptr, nullptr, b, nullptr, nullptr, nullptr, dlogits, 0, 1.0f, 0, st));
  }
  return BTX_OK;
}

// Scratch of btx_lb_loss_noalloc.  In host code this name is only a handle for
// cudaGetSymbolAddress; the device address it resolves to differs per GPU.
static __device__ __align__(256) unsigned char g_lb_noalloc_scratch[BTX_LB_NOALLOC_SCRATCH_BYTES];

static btx_status lb_noalloc_scratch(void** out) {
  constexpr int kMaxDevices = 64;
  static std::mutex mu;
  static void* addr[kMaxDevices] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return BTX_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return BTX_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(mu);
  if (addr[dev] == nullptr) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_lb_noalloc_scratch) != cudaSuccess || ptr == nullptr) return BTX_ERR_CUDA;
    addr[dev] = ptr;
  }
  *out = addr[dev];
  return BTX_OK;
}

extern "C" btx_status btx_lb_loss_noalloc(const btx_moe_desc* desc, const float* logits, const float* router_bias,
                                          float* loss, float* u, float* p, float* dlogits, void* stream) {
  Plan pl;
  btx_status s = lb_loss_validate(desc, logits, loss, u, p, &pl);
  if (s != BTX_OK) return s;
  if (pl.workspace_bytes > (size_t)BTX_LB_NOALLOC_SCRATCH_BYTES) return BTX_ERR_WORKSPACE;   // beyond the static array
  void* scratch = nullptr;
  if ((s = lb_noalloc_scratch(&scratch)) != BTX_OK) return s;
  // btx_lb_loss clears the status block at the head of the scratch and overwrites every other
  // region before reading it, so stale contents of an earlier call are harmless.
  return btx_lb_loss(desc, logits, router_bias, loss, u, p, dlogits, scratch, BTX_LB_NOALLOC_SCRATCH_BYTES, stream);
}

extern "C" btx_status btx_device_status(const void* workspace, void* stream, int32_t* device_status) {
  if (!workspace || !device_status) return BTX_ERR_INVALID_ARG;
  int32_t word = 0;
  cudaStream_t st = (cudaStream_t)stream;
  if (cudaMemcpyAsync(&word, workspace, 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return BTX_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return BTX_ERR_CUDA;
  *device_status = word == 0 ? BTX_OK : BTX_ERR_TIMEOUT;
  return BTX_OK;
}

extern "C" btx_status btx_selftest_wait_expiry(void* workspace, size_t workspace_bytes, void* stream) {
  if (!workspace || misaligned(workspace)) return BTX_ERR_INVALID_ARG;
  if (workspace_bytes < (size_t)kStatusWords * 4) return BTX_ERR_WORKSPACE;
  btx_status s = check_device();
  if (s != BTX_OK) return s;
  cudaStream_t st = (cudaStream_t)stream;
  BTX_CUDA_OK(cudaMemsetAsync(workspace, 0, kStatusWords * 4, st));
  BTX_CUDA_OK(launch_wait_expiry_selftest((int32_t*)workspace, st));
  return BTX_OK;
}

extern "C" const char* btx_status_string(btx_status s) {
  switch (s) {
    case BTX_OK: return "ok";
    case BTX_ERR_INVALID_ARG: return "invalid argument";
    case BTX_ERR_UNSUPPORTED: return "unsupported configuration";
    case BTX_ERR_WORKSPACE: return "workspace or saved buffer too small";
    case BTX_ERR_ARCH: return "device is not compute capability 10.x";
    case BTX_ERR_CUDA: return "CUDA call failed";
    case BTX_ERR_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown status";
}

extern "C" int32_t btx_version(void) { return 100; }
