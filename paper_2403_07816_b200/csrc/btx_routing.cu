// Router, load-balancing loss, token permutation, row gather / combine and router backward.
// These are the bandwidth- and latency-bound steps around the expert GEMMs.
//
//   router      logits = W_l x (Section 3.2; BF16: on the tensor cores), top-k by repeated arg-max with
//               ties to the lower index, gate softmax over the selected logits, full softmax, partial
//               sums for the batch means u and p of Section 3.3; the last block to finish forms
//               u, p and L_LB = alpha E sum_i u_i p_i
//   permutation histogram -> exclusive scan -> stable scatter of the R assignments into
//               (expert ascending, token ascending) order; expert segments padded to whole 256-row tiles
//   gather      rows of x (or dy) copied into the padded expert-sorted layout
//   combine     y_t = sum over slots of the gate-scaled expert rows
//   router bwd  d logits from d gates and the two L_LB terms; dW_l = dz^T x; dx += W_l^T dz
#include "btx_route_dev.cuh"

namespace btx {

namespace {

using namespace routedev;

constexpr int kRouterThreads = 256;
constexpr int kRouterWarps = kRouterThreads / 32;
constexpr int kPermThreads = 256;
constexpr int kPermChunk = 1024;      // assignments per block of the permutation kernels

// ---------------------------------------------------------------------------------------------
// Router
// ---------------------------------------------------------------------------------------------
// Logits of up to four tokens t0 .. t0+nt-1 by one warp: every lane takes each 32nd 16-byte vector of the rows,
// so one fetch of a router row vector serves four tokens.  With WS the router rows come from shared memory as
// fp32, laid out [expert][quad of the vector][vector][4] so that the lanes of a warp read consecutive 16-byte
// words; otherwise from global memory through L1.  z: the warp's shared scratch, kMaxExperts floats per token.
constexpr int kRouteTokens = 4;
template <typename T, bool WS>
__device__ __forceinline__ void route_logits4(int t0, int nt, int d, int E, const T* __restrict__ x,
                                              const T* __restrict__ wr, const float* ws, const float* __restrict__ bias,
                                              const float* __restrict__ given_logits, float (*z)[kMaxExperts], int lane) {
  constexpr int VN = Vec<T>::N, NT = kRouteTokens;
  if (given_logits != nullptr) {
    for (int e = lane; e < E; e += 32) {
      const float b = bias ? bias[e] : 0.f;
      for (int i = 0; i < nt; ++i) z[i][e] = given_logits[(size_t)(t0 + i) * E + e] + b;
    }
    return;
  }
  const T* xr[NT];
#pragma unroll
  for (int i = 0; i < NT; ++i) xr[i] = x + (size_t)(t0 + min(i, nt - 1)) * d;   // absent tokens repeat the last one
  const int vecs = d / VN;
  for (int eb = 0; eb < E; eb += 8) {
    float acc[NT][8];
#pragma unroll
    for (int i = 0; i < NT; ++i)
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;
#pragma unroll 2
    for (int v = lane; v < vecs; v += 32) {
      uint4 q[NT];
#pragma unroll
      for (int i = 0; i < NT; ++i) q[i] = __ldcs(reinterpret_cast<const uint4*>(xr[i]) + v);   // streamed once
      float u[NT][VN];
#pragma unroll
      for (int i = 0; i < NT; ++i) Vec<T>::unpack(q[i], u[i]);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        if (eb + j < E) {
          float wv[VN];
          if (WS) {
#pragma unroll
            for (int h = 0; h < VN / 4; ++h) {
              const float4 w4 = *reinterpret_cast<const float4*>(ws + (((size_t)(eb + j) * (VN / 4) + h) * vecs + v) * 4);
              wv[4 * h] = w4.x; wv[4 * h + 1] = w4.y; wv[4 * h + 2] = w4.z; wv[4 * h + 3] = w4.w;
            }
          } else {
            Vec<T>::load(wr + (size_t)(eb + j) * d + (size_t)v * VN, wv);
          }
#pragma unroll
          for (int i = 0; i < NT; ++i)
#pragma unroll
            for (int c = 0; c < VN; ++c) acc[i][j] = fmaf(u[i][c], wv[c], acc[i][j]);
        }
      }
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (eb + j < E) {
        const float b = bias ? bias[eb + j] : 0.f;
#pragma unroll
        for (int i = 0; i < NT; ++i) {
          float sum = acc[i][j];
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
          if (lane == 0) z[i][eb + j] = sum + b;
        }
      }
    }
  }
}

// BF16: logits of up to sixteen tokens t0 .. t0+nt-1 by one warp on the tensor cores (mma.sync m16n8k16, fp32
// accumulation): tokens are the rows, eight experts the columns.  Lane (g, tg) = (lane / 4, lane % 4) loads 16
// bytes of rows g and g + 8 of x and of router row g at columns c0 + 8 tg, and feeds them to two MMAs as the
// contraction slots its registers stand for; the order of the contraction index inside an MMA is free as long
// as both operands use the same one, so nothing is shuffled or staged.  A warp instruction reads 64
// contiguous bytes of each of 8 rows (whole sectors), x is streamed past L1, the 32 KB of router rows stay
// in it.  A block takes sixteen tokens at a time and its eight warps an eighth of the columns each (short load
// chains, a block per 16 tokens to spread over the multiprocessors); the partial sums meet in shared memory
// and are added in warp order.  About 70 instructions per token instead of 1800 with FMAs.
constexpr int kRouteMmaTokens = 16;
__device__ __forceinline__ void mma_bf16_16x8x16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                                 uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// Partial logits over the column blocks c_begin, c_begin + c_step, ... (32 columns each) of tokens t0 ..
// t0+nt-1 and experts eb .. eb+7.  c[0], c[1]: token g, experts eb + 2 tg, + 1; c[2], c[3]: token g + 8.
__device__ __forceinline__ void route_mma_partial(int t0, int nt, int d, int E, int eb, int c_begin, int c_step,
                                                  const __nv_bfloat16* __restrict__ x,
                                                  const __nv_bfloat16* __restrict__ wr, int lane, float (&c)[4]) {
  const int g = lane >> 2, tg = lane & 3;
  const __nv_bfloat16* x0 = x + (size_t)(t0 + min(g, nt - 1)) * d;        // absent tokens repeat the last one
  const __nv_bfloat16* x1 = x + (size_t)(t0 + min(g + 8, nt - 1)) * d;
  const __nv_bfloat16* w = wr + (size_t)min(eb + g, E - 1) * d;            // absent experts repeat the last one
#pragma unroll
  for (int i = 0; i < 4; ++i) c[i] = 0.f;
  // the trip count is the same for all lanes (the MMAs need the whole warp); a lane whose 8 columns lie past
  // the end of the rows (d is a multiple of 8, not necessarily of 32) contributes zeros
#pragma unroll 4
  for (int cb = c_begin; cb < d; cb += c_step) {
    const int c0 = cb + tg * 8;
    uint4 lo = make_uint4(0, 0, 0, 0), hi = lo, b = lo;
    if (c0 < d) {
      lo = __ldcs(reinterpret_cast<const uint4*>(x0 + c0));
      hi = __ldcs(reinterpret_cast<const uint4*>(x1 + c0));
      b = __ldg(reinterpret_cast<const uint4*>(w + c0));
    }
    mma_bf16_16x8x16(c, lo.x, hi.x, lo.y, hi.y, b.x, b.y);
    mma_bf16_16x8x16(c, lo.z, hi.z, lo.w, hi.w, b.z, b.w);
  }
}

// Stores the (unperturbed) logits of token t, adds the Sample Top-1 noise, and routes: top-k by repeated
// arg-max with ties to the lower index, gates, full softmax.  On return lane l holds the dense gate and the
// probability of experts l and l + 32.
__device__ __forceinline__ void route_finish_token(int t, int E, int k, int routing, const float* __restrict__ noise,
                                                   float inv_tau, float* z, int lane, float* __restrict__ logits,
                                                   int32_t* __restrict__ topk, float* __restrict__ gates,
                                                   float* __restrict__ probs, float (&my_g)[2], float (&my_p)[2]) {
  for (int e = lane; e < E; e += 32) {
    logits[(size_t)t * E + e] = z[e];                             // reported logits are unperturbed
    if (noise != nullptr) z[e] = z[e] + noise[(size_t)t * E + e]; // one fp32 addition decides the expert
  }
  __syncwarp();
  route_select(t, E, k, routing, noise != nullptr ? inv_tau : 1.0f, z, lane, topk, gates, probs, my_g, my_p);
}

// u, p and L_LB = alpha E sum_i u_i p_i from the per-block partial sums, by one block of 256 threads: one warp
// per (expert, u|p) pair, lanes sum strided block partials in double, then a fixed-order shuffle tree, so the
// result does not depend on scheduling.
__device__ __forceinline__ void lb_finalize(int Tn, int E, int nblocks, float alpha, const float* route_part,
                                            float* __restrict__ u, float* __restrict__ p, float* __restrict__ loss,
                                            double* __restrict__ up64) {
  __shared__ double su[kMaxExperts], sp[kMaxExperts];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int pair = warp; pair < 2 * E; pair += kRouterWarps) {
    double s = 0.0;
    for (int b0 = lane; b0 < nblocks; b0 += 8 * 32) {     // eight loads ahead, added in the same order as one by one
      float v[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] = b0 + i * 32 < nblocks ? __ldcg(route_part + (size_t)(b0 + i * 32) * 2 * E + pair) : 0.f;
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if (b0 + i * 32 < nblocks) s += (double)v[i];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    s /= (double)Tn;
    if (lane == 0) {
      if (pair & 1) { sp[pair >> 1] = s; p[pair >> 1] = (float)s; up64[E + (pair >> 1)] = s; }
      else { su[pair >> 1] = s; u[pair >> 1] = (float)s; up64[pair >> 1] = s; }
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    double acc = 0.0;
    for (int e = 0; e < E; ++e) acc += su[e] * sp[e];
    loss[0] = (float)((double)alpha * (double)E * acc);
  }
}

// One warp per four tokens; the blocks are persistent (two per multiprocessor) and, when the router matrix fits
// (E*d fp32 values in at most 64 KB), keep it in shared memory as fp32, so the inner loop neither fetches nor
// converts router rows per token.  Every block leaves its partial sums of the gates and probabilities; the
// block that finishes last (a ticket in the workspace status block, zero when the kernel starts) forms the
// batch means and the loss from all of them.
template <typename T, bool WS, bool MMA>
__global__ void __launch_bounds__(kRouterThreads, MMA ? 4 : 2)
router_kernel(int Tn, int d, int E, int k, int routing, float alpha, const T* __restrict__ x, const T* __restrict__ wr,
              const float* __restrict__ bias, const float* __restrict__ given_logits,
              const float* __restrict__ noise, float inv_tau,
              float* __restrict__ logits, int32_t* __restrict__ topk, float* __restrict__ gates,
              float* __restrict__ probs, float* route_part, float* __restrict__ u, float* __restrict__ p,
              float* __restrict__ loss, double* __restrict__ up64, int32_t* ticket) {
  extern __shared__ __align__(16) float ws[];             // WS: the router rows as fp32
  constexpr int NTOK = MMA ? kRouteMmaTokens : kRouteTokens;             // tokens a warp routes at a time
  __shared__ float zs[MMA ? 1 : kRouterWarps][NTOK][kMaxExperts];
  __shared__ float part[MMA ? kRouterWarps : 1][kRouteMmaTokens][8];      // MMA: partial logits of the warps
  __shared__ float red[kRouterWarps][kMaxExperts][2];
  __shared__ int is_last;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  allow_dependents();
  if (WS) {
    constexpr int VN = Vec<T>::N;
    const int vecs = d / VN;
    for (int idx = threadIdx.x; idx < E * d; idx += kRouterThreads) {
      const int e = idx / d, c = idx - e * d, v = c / VN, r = c - v * VN;
      ws[(((size_t)e * (VN / 4) + r / 4) * vecs + v) * 4 + (r & 3)] = to_f32(wr[idx]);
    }
    __syncthreads();
  }
  float u_acc[2] = {0.f, 0.f}, p_acc[2] = {0.f, 0.f};   // lane l accumulates experts l and l + 32 over this warp's tokens
  const float scale = noise != nullptr ? inv_tau : 1.0f;
  if constexpr (MMA) {
    // ---- BF16: a block per sixteen tokens, the columns split over its warps ----
    for (int grp = blockIdx.x; grp * NTOK < Tn; grp += gridDim.x) {
      const int t = grp * NTOK, nt = min(NTOK, Tn - t);
      for (int eb = 0; eb < E; eb += 8) {
        float c[4];
        route_mma_partial(t, nt, d, E, eb, warp * 32, kRouterWarps * 32, x, wr, lane, c);
        const int g = lane >> 2, tg = lane & 3;
        part[warp][g][2 * tg] = c[0]; part[warp][g][2 * tg + 1] = c[1];
        part[warp][g + 8][2 * tg] = c[2]; part[warp][g + 8][2 * tg + 1] = c[3];
        __syncthreads();
        if (threadIdx.x < NTOK * 8) {
          const int tok = threadIdx.x >> 3, e = eb + (threadIdx.x & 7);
          if (e < E) {
            float a = 0.f;
            for (int w = 0; w < kRouterWarps; ++w) a += part[w][tok][threadIdx.x & 7];
            zs[0][tok][e] = a + (bias ? bias[e] : 0.f);
          }
        }
        __syncthreads();
      }
      // few experts: several tokens are routed side by side, one lane per (token, expert); the passes go to
      // different warps
      if (E <= 4) {
        if (warp * 8 < nt)
          route_select_group<4>(t, warp * 8, nt, E, k, routing, scale, noise, zs[0], lane, logits, topk, gates, probs, u_acc[0], p_acc[0]);
      } else if (E <= 8) {
        if (warp * 4 < nt)
          route_select_group<8>(t, warp * 4, nt, E, k, routing, scale, noise, zs[0], lane, logits, topk, gates, probs, u_acc[0], p_acc[0]);
      } else if (E <= 16) {
        if (warp * 2 < nt)
          route_select_group<16>(t, warp * 2, nt, E, k, routing, scale, noise, zs[0], lane, logits, topk, gates, probs, u_acc[0], p_acc[0]);
      } else {
        for (int i = warp; i < nt; i += kRouterWarps) {
          float my_g[2], my_p[2];
          route_finish_token(t + i, E, k, routing, noise, inv_tau, zs[0][i], lane, logits, topk, gates, probs, my_g, my_p);
#pragma unroll
          for (int h = 0; h < 2; ++h) { u_acc[h] += my_g[h]; p_acc[h] += my_p[h]; }
        }
      }
      __syncthreads();                                    // zs is written again for the next sixteen tokens
    }
  } else {
    // ---- FP32 (or given logits): a warp per four tokens ----
    for (int t = (blockIdx.x * kRouterWarps + warp) * NTOK; t < Tn; t += gridDim.x * kRouterWarps * NTOK) {
      const int nt = min(NTOK, Tn - t);
      route_logits4<T, WS>(t, nt, d, E, x, wr, ws, bias, given_logits, zs[warp], lane);
      __syncwarp();
      if (E <= 4) {
        route_select_group<4>(t, 0, nt, E, k, routing, scale, noise, zs[warp], lane, logits, topk, gates, probs, u_acc[0], p_acc[0]);
      } else if (E <= 8) {
        route_select_group<8>(t, 0, nt, E, k, routing, scale, noise, zs[warp], lane, logits, topk, gates, probs, u_acc[0], p_acc[0]);
      } else if (E <= 16) {
        for (int i0 = 0; i0 < nt; i0 += 2)
          route_select_group<16>(t, i0, nt, E, k, routing, scale, noise, zs[warp], lane, logits, topk, gates, probs, u_acc[0], p_acc[0]);
      } else {
        for (int i = 0; i < nt; ++i) {
          float my_g[2], my_p[2];
          route_finish_token(t + i, E, k, routing, noise, inv_tau, zs[warp][i], lane, logits, topk, gates, probs, my_g, my_p);
#pragma unroll
          for (int h = 0; h < 2; ++h) { u_acc[h] += my_g[h]; p_acc[h] += my_p[h]; }
        }
      }
    }
  }
#pragma unroll
  for (int h = 0; h < 2; ++h)
    if (lane + 32 * h < E) { red[warp][lane + 32 * h][0] = u_acc[h]; red[warp][lane + 32 * h][1] = p_acc[h]; }
  __syncthreads();
  if (threadIdx.x < 2 * E) {
    int e = threadIdx.x >> 1, which = threadIdx.x & 1;
    float s = 0.f;
    for (int w = 0; w < kRouterWarps; ++w) s += red[w][e][which];
    route_part[(size_t)blockIdx.x * 2 * E + threadIdx.x] = s;
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) is_last = (atomicAdd(ticket, 1) == (int)gridDim.x - 1);
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  lb_finalize(Tn, E, (int)gridDim.x, alpha, route_part, u, p, loss, up64);
}

// ---------------------------------------------------------------------------------------------
// Permutation
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kPermThreads)
perm_count_kernel(int R, int E, int nblocks, const int32_t* __restrict__ topk, int32_t* __restrict__ perm_counts) {
  __shared__ int hist[kMaxExperts];
  allow_dependents();
  if (threadIdx.x < kMaxExperts) hist[threadIdx.x] = 0;
  __syncthreads();
  grid_dependency_wait();
  int base = blockIdx.x * kPermChunk;
  int end = min(R, base + kPermChunk);
  for (int i = base + threadIdx.x; i < end; i += kPermThreads) atomicAdd(&hist[topk[i]], 1);
  __syncthreads();
  if (threadIdx.x < E) perm_counts[threadIdx.x * nblocks + blockIdx.x] = hist[threadIdx.x];
}

__global__ void perm_scan_kernel(int E, int nblocks, int mt_max, int cap, const int32_t* __restrict__ perm_counts,
                                 int32_t* __restrict__ perm_base, int32_t* __restrict__ counts,
                                 int32_t* __restrict__ offsets, int32_t* __restrict__ pad_offsets,
                                 int32_t* __restrict__ tile_expert) {
  __shared__ int scnt[kMaxExperts];
  __shared__ int spad[kMaxExperts + 1];
  int tid = threadIdx.x;
  allow_dependents();
  grid_dependency_wait();
  if (tid < E) {
    int run = 0;
    for (int b = 0; b < nblocks; ++b) {
      perm_base[tid * nblocks + b] = run;
      run += perm_counts[tid * nblocks + b];
    }
    run = min(run, cap);               // rows kept under the capacity limit
    scnt[tid] = run;
    counts[tid] = run;
  }
  __syncthreads();
  if (tid == 0) {
    int o = 0, po = 0;
    for (int e = 0; e < E; ++e) {
      offsets[e] = o; pad_offsets[e] = po; spad[e] = po;
      o += scnt[e];
      po += (scnt[e] + kRowTile - 1) / kRowTile * kRowTile;
    }
    offsets[E] = o; pad_offsets[E] = po; spad[E] = po;
  }
  __syncthreads();
  for (int mt = tid; mt < mt_max; mt += blockDim.x) {
    int row = mt * kRowTile, ex = -1;
    for (int e = 0; e < E; ++e)
      if (row >= spad[e] && row < spad[e + 1]) ex = e;
    tile_expert[mt] = ex;
  }
}

__global__ void __launch_bounds__(kPermThreads)
perm_scatter_kernel(int R, int E, int nblocks, int cap, int r_pad_max, const int32_t* __restrict__ topk,
                    const int32_t* __restrict__ perm_base, const int32_t* __restrict__ counts,
                    const int32_t* __restrict__ offsets, const int32_t* __restrict__ pad_offsets,
                    int32_t* __restrict__ perm, int32_t* __restrict__ inv_perm, int32_t* __restrict__ rowmap,
                    int32_t* __restrict__ flat2row) {
  constexpr int NW = kPermThreads / 32;
  __shared__ int running[kMaxExperts + 1];
  __shared__ int wcnt[NW][kMaxExperts + 1];
  __shared__ int spad[kMaxExperts + 1], scnt[kMaxExperts];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  allow_dependents();
  grid_dependency_wait();
  if (threadIdx.x < E) running[threadIdx.x] = perm_base[threadIdx.x * nblocks + blockIdx.x];
  if (threadIdx.x <= E) spad[threadIdx.x] = pad_offsets[threadIdx.x];
  if (threadIdx.x < E) scnt[threadIdx.x] = counts[threadIdx.x];
  __syncthreads();
  // padding rows (behind an expert's last real row, and behind the last expert) map to no assignment;
  // the real rows are written below, by whichever block holds their assignment
  for (int rp = blockIdx.x * kPermThreads + threadIdx.x; rp < r_pad_max; rp += gridDim.x * kPermThreads) {
    bool real = false;
    for (int e = 0; e < E; ++e)
      if (rp >= spad[e] && rp < spad[e] + scnt[e]) real = true;
    if (!real) rowmap[rp] = -1;
  }
  const int base = blockIdx.x * kPermChunk;
  const int end = min(R, base + kPermChunk);
  for (int r0 = base; r0 < end; r0 += kPermThreads) {
    for (int j = threadIdx.x; j < NW * (kMaxExperts + 1); j += kPermThreads) (&wcnt[0][0])[j] = 0;
    __syncthreads();
    int i = r0 + threadIdx.x;
    int e = (i < end) ? topk[i] : E;                 // E = dummy bucket for idle lanes
    unsigned same = __match_any_sync(0xffffffffu, e);
    int rank = __popc(same & ((1u << lane) - 1u));
    if (rank == 0) wcnt[warp][e] = __popc(same);
    __syncthreads();
    if (i < end) {
      int before = 0;
      for (int w = 0; w < warp; ++w) before += wcnt[w][e];
      int within = running[e] + before + rank;       // stable rank inside the expert
      if (within < cap) {
        int r = offsets[e] + within;                 // tight sorted row
        int rp = pad_offsets[e] + within;            // padded sorted row
        perm[r] = i;
        inv_perm[i] = r;
        rowmap[rp] = i;
        flat2row[i] = rp;
      } else {                                       // beyond the expert's capacity: dropped
        inv_perm[i] = -1;
        flat2row[i] = -1;
      }
    }
    __syncthreads();
    if (threadIdx.x < E) {
      int s = 0;
      for (int w = 0; w < NW; ++w) s += wcnt[w][threadIdx.x];
      running[threadIdx.x] += s;
    }
    __syncthreads();
  }
}

// ---------------------------------------------------------------------------------------------
// Small batches (R = T*k <= 1024, e.g. decoding): router, loss and permutation in ONE launch
// instead of six.  (The workspace status block is zeroed at the start of every forward call; its
// word 8 is the ticket counter.)
// ---------------------------------------------------------------------------------------------
// One block per token computes its logits (eight warps share the row) and routes it; the block that
// finishes last (a ticket counter in the workspace status block) then forms u, p, the loss and the
// permutation.  Every sum runs in a fixed order, so results do not depend on which block is last.
template <typename T>
__global__ void __launch_bounds__(kSmallThreads)
route_permute_small_kernel(int Tn, int d, int E, int k, int routing, float alpha, int mt_max, int r_pad_max, int cap,
                           const T* __restrict__ x, const T* __restrict__ wr, const float* __restrict__ bias,
                           const float* __restrict__ noise, float inv_tau, float* logits, int32_t* topk, float* gates, float* probs, float* __restrict__ u,
                           float* __restrict__ p, double* __restrict__ up64, float* __restrict__ loss,
                           int32_t* __restrict__ counts,
                           int32_t* __restrict__ offsets, int32_t* __restrict__ pad_offsets,
                           int32_t* __restrict__ tile_expert, int32_t* __restrict__ perm,
                           int32_t* __restrict__ inv_perm, int32_t* __restrict__ rowmap,
                           int32_t* __restrict__ flat2row, int32_t* ticket) {
  constexpr int NW = kSmallThreads / 32;
  __shared__ float part[NW][kMaxExperts];
  __shared__ float z[kMaxExperts];
  __shared__ int is_last;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t = blockIdx.x;
  allow_dependents();

  token_logit_parts<T>(x + (size_t)t * d, wr, d, E, warp, lane, part);
  __syncthreads();
  if (threadIdx.x < E) {
    float a = 0.f;
    for (int w = 0; w < NW; ++w) a += part[w][threadIdx.x];
    a += bias ? bias[threadIdx.x] : 0.f;
    logits[(size_t)t * E + threadIdx.x] = a;                      // reported logits are unperturbed
    if (noise != nullptr) a = a + noise[(size_t)t * E + threadIdx.x];   // one fp32 addition decides the expert
    z[threadIdx.x] = a;
  }
  __syncthreads();
  if (warp == 0) {
    float my_g[2], my_p[2];
    route_select(t, E, k, routing, noise != nullptr ? inv_tau : 1.0f, z, lane, topk, gates, probs, my_g, my_p);
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) is_last = (atomicAdd(ticket, 1) == (int)gridDim.x - 1);
  __syncthreads();
  if (!is_last) return;
  __threadfence();

  small_batch_finish<kSmallThreads>((int)threadIdx.x, [] { __syncthreads(); }, Tn, E, k, alpha, mt_max, r_pad_max, cap, topk,
                                    gates, probs, u, p, up64, loss, counts, offsets, pad_offsets, tile_expert, perm,
                                    inv_perm, rowmap, flat2row);
}

// ---------------------------------------------------------------------------------------------
// Gather into the padded sorted layout, combine out of it
// ---------------------------------------------------------------------------------------------
// A warp per token: the row is read once (eight 16-byte loads in flight per lane) and written to the sorted row
// of each of its k assignments (none for a dropped one); then a warp per padding row writes zeros.
__global__ void __launch_bounds__(256)
gather_rows_kernel(int Tn, int k, int row_vecs, const uint4* __restrict__ src, uint4* __restrict__ dst,
                   const int32_t* __restrict__ rowmap, const int32_t* __restrict__ flat2row,
                   const int32_t* __restrict__ pad_offsets, int E) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  allow_dependents();
  grid_dependency_wait();
  for (int t = blockIdx.x * 8 + warp; t < Tn; t += gridDim.x * 8) {
    const uint4* s = src + (size_t)t * row_vecs;
    for (int c0 = lane; c0 < row_vecs; c0 += 8 * 32) {
      uint4 q[8];
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if (c0 + i * 32 < row_vecs) q[i] = __ldcs(s + c0 + i * 32);
      for (int sl = 0; sl < k; ++sl) {
        const int rp = flat2row[(size_t)t * k + sl];
        if (rp < 0) continue;
        uint4* o = dst + (size_t)rp * row_vecs;
#pragma unroll
        for (int i = 0; i < 8; ++i)
          if (c0 + i * 32 < row_vecs) o[c0 + i * 32] = q[i];
      }
    }
  }
  const int total = pad_offsets[E];
  for (int rp = blockIdx.x * 8 + warp; rp < total; rp += gridDim.x * 8) {
    if (rowmap[rp] >= 0) continue;
    uint4* o = dst + (size_t)rp * row_vecs;
    for (int c = lane; c < row_vecs; c += 32) o[c] = make_uint4(0, 0, 0, 0);
  }
}

template <typename T> __device__ __forceinline__ void store4(T* p, float4 v);
template <> __device__ __forceinline__ void store4<float>(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }
template <> __device__ __forceinline__ void store4<__nv_bfloat16>(__nv_bfloat16* p, float4 v) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
  uint2 q;
  q.x = *reinterpret_cast<uint32_t*>(&a);
  q.y = *reinterpret_cast<uint32_t*>(&b);
  *reinterpret_cast<uint2*>(p) = q;
}

// y[t, :] = sum_slot sum_split rows[split][t*k + slot, :]   (+ sum_e dz[t,e] * wr[e, :] when dz != nullptr)
// `kept` (optional): flat assignment -> sorted row; a negative entry is a dropped assignment, whose
// row was never written and counts as zero.  A thread owns 16 bytes of the output row (8 columns in BF16,
// 4 in FP32), so in BF16 it has two 16-byte loads in flight per slot and stores one whole vector.
template <typename T>
__global__ void __launch_bounds__(256)
combine_kernel(int Tn, int d, int k, int E, int splits, const float* __restrict__ rows, const float* __restrict__ dz,
               const T* __restrict__ wr, const int32_t* __restrict__ kept, T* __restrict__ y) {
  constexpr int G = Vec<T>::N / 4;                        // float4 groups per thread
  const size_t split_stride = (size_t)Tn * k * d;
  const int vecs = d / Vec<T>::N;
  allow_dependents();
  grid_dependency_wait();
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < (size_t)Tn * vecs;
       i += (size_t)gridDim.x * blockDim.x) {
    const int t = (int)(i / vecs), c = (int)(i % vecs) * Vec<T>::N;
    float4 acc[G];
#pragma unroll
    for (int g = 0; g < G; ++g) acc[g] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s = 0; s < k; ++s) {
      if (kept != nullptr && kept[(size_t)t * k + s] < 0) continue;
      for (int sp = 0; sp < splits; ++sp) {
        const float* r = rows + sp * split_stride + ((size_t)t * k + s) * d + c;
        float4 v[G];
#pragma unroll
        for (int g = 0; g < G; ++g) v[g] = *reinterpret_cast<const float4*>(r + 4 * g);
#pragma unroll
        for (int g = 0; g < G; ++g) { acc[g].x += v[g].x; acc[g].y += v[g].y; acc[g].z += v[g].z; acc[g].w += v[g].w; }
      }
    }
    if (dz != nullptr) {
      for (int e = 0; e < E; ++e) {
        const float gz = dz[(size_t)t * E + e];
        float wv[Vec<T>::N];
        Vec<T>::load(wr + (size_t)e * d + c, wv);
#pragma unroll
        for (int g = 0; g < G; ++g) {
          acc[g].x = fmaf(gz, wv[4 * g], acc[g].x); acc[g].y = fmaf(gz, wv[4 * g + 1], acc[g].y);
          acc[g].z = fmaf(gz, wv[4 * g + 2], acc[g].z); acc[g].w = fmaf(gz, wv[4 * g + 3], acc[g].w);
        }
      }
    }
    if (G == 1) {
      store4<T>(y + (size_t)t * d + c, acc[0]);
    } else {
      float f[8] = {acc[0].x, acc[0].y, acc[0].z, acc[0].w, acc[G - 1].x, acc[G - 1].y, acc[G - 1].z, acc[G - 1].w};
      __nv_bfloat162 h[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) h[j] = __floats2bfloat162_rn(f[2 * j], f[2 * j + 1]);
      *reinterpret_cast<uint4*>(y + (size_t)t * d + c) = *reinterpret_cast<uint4*>(h);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Router backward
// ---------------------------------------------------------------------------------------------
// Row-dot partials of the dgrad-2 epilogue, [column tile][padded row]: summed over the column tiles in
// tile order, one thread per padded row (consecutive rows, so every load is coalesced), into tile 0.
__global__ void __launch_bounds__(256)
dg_rowsum_kernel(int nt, int r_pad_max, int E, const int32_t* __restrict__ pad_offsets, float* __restrict__ dg_part) {
  const int rp = blockIdx.x * blockDim.x + threadIdx.x;
  if (rp >= pad_offsets[E]) return;
  float a = 0.f;
#pragma unroll 8
  for (int n = 0; n < nt; ++n) a += dg_part[(size_t)n * r_pad_max + rp];
  dg_part[rp] = a;
}

// One thread per token: d gate of every slot (the summed row-dot of its row plus the u-term of L_LB),
// then the softmax Jacobians and the p-term of L_LB.  The L_LB terms are differences of nearly equal
// numbers when the load is balanced (c_i - sum_j p_j c_j with all c_i close to one another, and
// g_a (dg_a - sum_j g_j dg_j) with all dg_j close), which multiplies any error in sum_j p_j = 1 and
// sum_j g_j = 1 a hundredfold: the thread therefore forms the two softmaxes again, in double, from the
// saved fp32 logits (`logits` non-null; for Sample Top-1, whose softmax is that of the perturbed logits
// and which has no L_LB terms, it takes the stored fp32 values), uses the batch means kept in double,
// and rounds the result to fp32 once.
__global__ void __launch_bounds__(64)
router_dz_kernel(int Tn, int E, int k, int routing, float alpha, float lb_scale, int stopgrad_u,
                 const int32_t* __restrict__ topk, const float* __restrict__ gates,
                 const float* __restrict__ probs, const float* __restrict__ logits,
                 const double* __restrict__ up64,
                 const int32_t* __restrict__ flat2row, const float* __restrict__ dg_part, float dz_scale,
                 float* __restrict__ dz_out, float* __restrict__ dz_out2) {
  int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= Tn) return;
  const double* u = up64;
  const double* p = up64 + E;
  double pt[kMaxExperts], dzv[kMaxExperts], gt[kMaxExperts], dg[kMaxExperts];
  if (logits != nullptr) {
    const float* z = logits + (size_t)t * E;
    double zmax = (double)z[0];
    for (int e = 1; e < E; ++e) zmax = fmax(zmax, (double)z[e]);
    double sum = 0.0;
    for (int e = 0; e < E; ++e) { pt[e] = exp((double)z[e] - zmax); sum += pt[e]; }
    for (int e = 0; e < E; ++e) pt[e] /= sum;
    if (routing == BTX_ROUTE_SWITCH) {
      gt[0] = pt[topk[t]];
    } else {
      double gsum = 0.0;
      for (int s = 0; s < k; ++s) { gt[s] = exp((double)z[topk[(size_t)t * k + s]] - zmax); gsum += gt[s]; }
      for (int s = 0; s < k; ++s) gt[s] /= gsum;
    }
  } else {
    for (int e = 0; e < E; ++e) pt[e] = (double)probs[(size_t)t * E + e];
    for (int s = 0; s < k; ++s) gt[s] = (double)gates[(size_t)t * k + s];
  }
  for (int e = 0; e < E; ++e) dzv[e] = 0.0;
  const double lbc = (double)lb_scale * (double)alpha * (double)E / (double)Tn;
  for (int s = 0; s < k; ++s) {
    double a = 0.0;
    if (dg_part != nullptr) {
      int rp = flat2row[(size_t)t * k + s];
      if (rp >= 0) a = (double)dg_part[rp];          // a dropped assignment has no path into y
    }
    if (!stopgrad_u) a += lbc * p[topk[(size_t)t * k + s]];
    dg[s] = a;
  }
  if (routing == BTX_ROUTE_SWITCH) {
    int sel = topk[t];
    double ps = pt[sel];
    for (int e = 0; e < E; ++e) dzv[e] = -dg[0] * ps * pt[e];
    dzv[sel] += dg[0] * ps;
  } else {
    double inner = 0.0;
    for (int s = 0; s < k; ++s) inner += gt[s] * dg[s];
    for (int s = 0; s < k; ++s) dzv[topk[(size_t)t * k + s]] = gt[s] * (dg[s] - inner);
  }
  double pc = 0.0;
  for (int e = 0; e < E; ++e) pc += pt[e] * (lbc * u[e]);
  for (int e = 0; e < E; ++e) {
    float v = (float)((dzv[e] + pt[e] * (lbc * u[e] - pc)) * (double)dz_scale);
    dz_out[(size_t)t * E + e] = v;
    if (dz_out2 != nullptr) dz_out2[(size_t)t * E + e] = v;
  }
}

constexpr int kWrTokens = 128;   // tokens per chunk of the router-weight gradient

// partial[chunk][e][c] = sum over the chunk's tokens of dz[t,e] * x[t,c]; each thread owns one 16-byte
// vector of columns (8 in BF16, 4 in FP32) and four experts at a time.
template <typename T>
__global__ void __launch_bounds__(128)
router_dw_partial_kernel(int Tn, int d, int E, const T* __restrict__ x, const float* __restrict__ dz,
                         float* __restrict__ part, float* __restrict__ bias_part) {
  constexpr int VN = Vec<T>::N;
  __shared__ float sdz[kWrTokens * kMaxExperts];
  const int chunk = blockIdx.x;
  const int t0 = chunk * kWrTokens, t1 = min(Tn, t0 + kWrTokens);
  for (int i = threadIdx.x; i < (t1 - t0) * E; i += blockDim.x) sdz[i] = dz[(size_t)t0 * E + i];
  __syncthreads();
  const int c = (blockIdx.y * blockDim.x + threadIdx.x) * VN;
  if (blockIdx.y == 0 && threadIdx.x < E) {
    float s = 0.f;
    for (int t = 0; t < t1 - t0; ++t) s += sdz[t * E + threadIdx.x];
    bias_part[(size_t)chunk * E + threadIdx.x] = s;
  }
  if (c >= d) return;
  for (int eb = 0; eb < E; eb += 4) {
    float acc[4][VN];
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
      for (int v = 0; v < VN; ++v) acc[j][v] = 0.f;
#pragma unroll 4
    for (int t = t0; t < t1; ++t) {
      float xv[VN];
      Vec<T>::load(x + (size_t)t * d + c, xv);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (eb + j < E) {
          const float g = sdz[(t - t0) * E + eb + j];
#pragma unroll
          for (int v = 0; v < VN; ++v) acc[j][v] = fmaf(g, xv[v], acc[j][v]);
        }
      }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (eb + j < E) {
        float* o = part + ((size_t)chunk * E + eb + j) * d + c;
#pragma unroll
        for (int v = 0; v < VN; v += 4)
          *reinterpret_cast<float4*>(o + v) = make_float4(acc[j][v], acc[j][v + 1], acc[j][v + 2], acc[j][v + 3]);
      }
    }
  }
}

__global__ void __launch_bounds__(256)
router_dw_reduce_kernel(int d, int E, int chunks, const float* __restrict__ part, const float* __restrict__ bias_part,
                        float* __restrict__ dw_router, float* __restrict__ dbias, int accumulate) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < E * d) {
    float s = 0.f;
    for (int ch = 0; ch < chunks; ++ch) s += part[(size_t)ch * E * d + i];
    dw_router[i] = accumulate ? dw_router[i] + s : s;
  }
  if (dbias != nullptr && blockIdx.x == 0 && threadIdx.x < E) {
    float s = 0.f;
    for (int ch = 0; ch < chunks; ++ch) s += bias_part[(size_t)ch * E + threadIdx.x];
    dbias[threadIdx.x] = accumulate ? dbias[threadIdx.x] + s : s;
  }
}

}  // namespace

// ---------------------------------------------------------------------------------------------
// Launchers
// ---------------------------------------------------------------------------------------------
template <typename T, bool WS, bool MMA>
static cudaError_t launch_router_t(const Plan& pl, int routing, float alpha, const void* x, const void* w_router,
                                   const float* bias, const float* given_logits, const float* noise, float inv_tau,
                                   const Buffers& b, size_t smem, cudaStream_t st) {
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(router_kernel<T, WS, MMA>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  // the ticket of the last-block finalisation is word 8 of the status block, zeroed by the caller
  int blocks = pl.route_blocks;                           // (the plan's count bounds the partial-sum buffer)
  if (!MMA) blocks = min(blocks, (pl.T + kRouterWarps * kRouteTokens - 1) / (kRouterWarps * kRouteTokens));
  router_kernel<T, WS, MMA><<<blocks, kRouterThreads, smem, st>>>(
      pl.T, pl.d, pl.E, pl.k, routing, alpha, (const T*)x, (const T*)w_router, bias, given_logits, noise, inv_tau,
      b.logits, b.topk, b.gates, b.probs, b.route_part, b.u, b.p, b.loss, b.up64, b.status + 8);
  return cudaGetLastError();
}

cudaError_t launch_router(const Plan& pl, int dtype, int routing, float alpha, const void* x, const void* w_router,
                          const float* bias, const float* given_logits, const float* noise, float inv_tau,
                          const Buffers& b, cudaStream_t st) {
  const size_t smem = (size_t)pl.E * pl.d * sizeof(float);
  const bool in_smem = given_logits == nullptr && smem > 0 && smem <= 64 * 1024;
  if (dtype == BTX_BF16)          // BF16 activations: the logits come from the tensor cores
    return launch_router_t<__nv_bfloat16, false, true>(pl, routing, alpha, x, w_router, bias, given_logits, noise, inv_tau, b, 0, st);
  return in_smem ? launch_router_t<float, true, false>(pl, routing, alpha, x, w_router, bias, given_logits, noise, inv_tau, b, smem, st)
                 : launch_router_t<float, false, false>(pl, routing, alpha, x, w_router, bias, given_logits, noise, inv_tau, b, 0, st);
}

bool route_permute_small_fits(const Plan& pl) { return pl.R <= kSmallMaxR; }

cudaError_t launch_route_permute_small(const Plan& pl, int dtype, int routing, float alpha, const void* x,
                                       const void* w_router, const float* bias, const float* noise, float inv_tau,
                                       const Buffers& b, cudaStream_t st) {
  if (dtype == BTX_BF16)
    route_permute_small_kernel<__nv_bfloat16><<<pl.T, kSmallThreads, 0, st>>>(
        pl.T, pl.d, pl.E, pl.k, routing, alpha, pl.mt_max, pl.r_pad_max, pl.capacity, (const __nv_bfloat16*)x,
        (const __nv_bfloat16*)w_router, bias, noise, inv_tau, b.logits, b.topk, b.gates, b.probs, b.u, b.p, b.up64, b.loss, b.counts, b.offsets,
        b.pad_offsets, b.tile_expert, b.perm, b.inv_perm, b.rowmap, b.flat2row, b.status + 8);
  else
    route_permute_small_kernel<float><<<pl.T, kSmallThreads, 0, st>>>(
        pl.T, pl.d, pl.E, pl.k, routing, alpha, pl.mt_max, pl.r_pad_max, pl.capacity, (const float*)x,
        (const float*)w_router, bias,
        noise, inv_tau, b.logits, b.topk, b.gates, b.probs, b.u, b.p, b.up64, b.loss, b.counts, b.offsets, b.pad_offsets, b.tile_expert, b.perm,
        b.inv_perm, b.rowmap, b.flat2row, b.status + 8);
  return cudaGetLastError();
}

// The three kernels follow the router kernel as programmatic dependents of one another (each waits for the one
// before it prior to reading).  Under a capacity limit the caller has filled perm with -1 beforehand.
cudaError_t launch_permute(const Plan& pl, const Buffers& b, cudaStream_t st) {
  cudaError_t e = launch_after_predecessor(perm_count_kernel, dim3(pl.perm_blocks), dim3(kPermThreads), 0, st, true, pl.R,
                                           pl.E, pl.perm_blocks, (const int32_t*)b.topk, b.perm_counts);
  if (e != cudaSuccess) return e;
  e = launch_after_predecessor(perm_scan_kernel, dim3(1), dim3(256), 0, st, true, pl.E, pl.perm_blocks, pl.mt_max,
                               pl.capacity, (const int32_t*)b.perm_counts, b.perm_base, b.counts, b.offsets,
                               b.pad_offsets, b.tile_expert);
  if (e != cudaSuccess) return e;
  return launch_after_predecessor(perm_scatter_kernel, dim3(pl.perm_blocks), dim3(kPermThreads), 0, st, true, pl.R, pl.E,
                                  pl.perm_blocks, pl.capacity, pl.r_pad_max, (const int32_t*)b.topk,
                                  (const int32_t*)b.perm_base, (const int32_t*)b.counts, (const int32_t*)b.offsets,
                                  (const int32_t*)b.pad_offsets, b.perm, b.inv_perm, b.rowmap, b.flat2row);
}

cudaError_t launch_gather_rows(const Plan& pl, const void* src, void* dst_sorted, const Buffers& b, cudaStream_t st) {
  int row_vecs = pl.d * pl.esize / 16;
  int blocks = min(pl.r_pad_max / 8, sm_count() * 16);
  // the gather's launch overlaps the run of the kernel before it
  return launch_after_predecessor(gather_rows_kernel, dim3(blocks), dim3(256), 0, st, true, pl.T, pl.k, row_vecs,
                                  (const uint4*)src, (uint4*)dst_sorted, (const int32_t*)b.rowmap,
                                  (const int32_t*)b.flat2row, (const int32_t*)b.pad_offsets, pl.E);
}

cudaError_t launch_combine(const Plan& pl, int dtype, const float* rows, int splits, void* y, const Buffers& b,
                           cudaStream_t st) {
  size_t n = (size_t)pl.T * (pl.d / (dtype == BTX_BF16 ? 8 : 4));
  int blocks = (int)min((n + 255) / 256, (size_t)sm_count() * 32);
  const int32_t* kept = pl.capped ? b.flat2row : nullptr;
  if (dtype == BTX_BF16)
    return launch_after_predecessor(combine_kernel<__nv_bfloat16>, dim3(blocks), dim3(256), 0, st, true, pl.T,
                                    pl.d, pl.k, pl.E, splits, rows, (const float*)nullptr,
                                    (const __nv_bfloat16*)nullptr, kept, (__nv_bfloat16*)y);
  combine_kernel<float><<<blocks, 256, 0, st>>>(pl.T, pl.d, pl.k, pl.E, splits, rows, nullptr, nullptr, kept, (float*)y);
  return cudaGetLastError();
}

cudaError_t launch_router_backward(const Plan& pl, int dtype, int routing, float alpha, float lb_scale,
                                   int stopgrad_u, int have_dg, const void* x, const void* w_router, const Buffers& b,
                                   void* dx, float* dw_router, float* dbias, float* dlogits_out, int accumulate,
                                   float dz_scale, int perturbed, cudaStream_t st) {
  if (have_dg)
    dg_rowsum_kernel<<<(pl.r_pad_max + 255) / 256, 256, 0, st>>>(pl.nt_dact, pl.r_pad_max, pl.E, b.pad_offsets, b.dg_part);
  router_dz_kernel<<<(pl.T + 63) / 64, 64, 0, st>>>(pl.T, pl.E, pl.k, routing, alpha, lb_scale, stopgrad_u, b.topk,
                                                    b.gates, b.probs, perturbed ? nullptr : b.logits, b.up64, b.flat2row,
                                                    have_dg ? b.dg_part : nullptr, dz_scale, b.dz, dlogits_out);
  if (x == nullptr) return cudaGetLastError();     // loss-only gradient (btx_lb_loss)
  const int vn = dtype == BTX_BF16 ? 8 : 4;
  dim3 grid(pl.wr_chunks, (pl.d / vn + 127) / 128);
  float* bias_part = b.dwr_part + (size_t)pl.wr_chunks * pl.E * pl.d;
  size_t n = (size_t)pl.T * (pl.d / vn);
  int cblocks = (int)min((n + 255) / 256, (size_t)sm_count() * 32);
  const int32_t* kept = pl.capped ? b.flat2row : nullptr;
  if (dtype == BTX_BF16) {
    router_dw_partial_kernel<__nv_bfloat16><<<grid, 128, 0, st>>>(pl.T, pl.d, pl.E, (const __nv_bfloat16*)x, b.dz,
                                                                  b.dwr_part, bias_part);
    combine_kernel<__nv_bfloat16><<<cblocks, 256, 0, st>>>(pl.T, pl.d, pl.k, pl.E, 1, b.dxp, b.dz,
                                                           (const __nv_bfloat16*)w_router, kept, (__nv_bfloat16*)dx);
  } else {
    router_dw_partial_kernel<float><<<grid, 128, 0, st>>>(pl.T, pl.d, pl.E, (const float*)x, b.dz, b.dwr_part,
                                                          bias_part);
    combine_kernel<float><<<cblocks, 256, 0, st>>>(pl.T, pl.d, pl.k, pl.E, 1, b.dxp, b.dz, (const float*)w_router,
                                                   kept, (float*)dx);
  }
  router_dw_reduce_kernel<<<(pl.E * pl.d + 255) / 256, 256, 0, st>>>(pl.d, pl.E, pl.wr_chunks, b.dwr_part, bias_part,
                                                                     dw_router, dbias, accumulate);
  return cudaGetLastError();
}

}  // namespace btx
