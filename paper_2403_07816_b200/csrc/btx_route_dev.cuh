// Device functions of the router shared by the routing kernels (btx_routing.cu) and the one-kernel
// small-batch forward (btx_gemm_fused.cu): 16-byte vector loads, the selection / gate / softmax step of
// one token (Section 3.2: top-k, SoftMax over the selected logits), the logits of one token by eight warps,
// and the batch means, loss (Section 3.3) and permutation of a small batch by one group of threads.
#pragma once

#include "btx_common.cuh"

namespace btx {
namespace routedev {

template <typename T> struct Vec;     // 16-byte vectors of the element type
template <> struct Vec<float> {
  static constexpr int N = 4;
  static __device__ __forceinline__ void unpack(const uint4& q, float (&v)[4]) {
    v[0] = __uint_as_float(q.x); v[1] = __uint_as_float(q.y); v[2] = __uint_as_float(q.z); v[3] = __uint_as_float(q.w);
  }
  static __device__ __forceinline__ void load(const float* p, float (&v)[4]) {
    float4 q = *reinterpret_cast<const float4*>(p);
    v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
  }
};
template <> struct Vec<__nv_bfloat16> {
  static constexpr int N = 8;
  static __device__ __forceinline__ void unpack(const uint4& q, float (&v)[8]) {
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&q);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float2 f = __bfloat1622float2(h[i]);
      v[2 * i] = f.x; v[2 * i + 1] = f.y;
    }
  }
  static __device__ __forceinline__ void load(const __nv_bfloat16* p, float (&v)[8]) {
    uint4 q = *reinterpret_cast<const uint4*>(p);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&q);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float2 f = __bfloat1622float2(h[i]);
      v[2 * i] = f.x; v[2 * i + 1] = f.y;
    }
  }
};

// Selection, gates and softmax for one token from the logits z[0..E) in shared memory, by the 32 lanes of
// the calling warp together: lane l owns experts l and l + 32.  Top-k is k rounds of a warp arg-max over
// (value descending, index ascending), so ties go to the lower index; the sums of the two softmaxes run over
// the experts (resp. the slots) in ascending order, one addition at a time, so the result does not depend on
// how the lanes are laid out.  The experts are chosen on z as it stands; the softmaxes are those of
// z * scale (scale = 1 except for Sample Top-1, whose temperature must not touch the arg-max: a
// rounded product could merge two distinct perturbed logits into a tie).  On return lane l holds the
// dense gate and probability of experts l (index 0) and l + 32 (index 1).
__device__ __forceinline__ void route_select(int t, int E, int k, int routing, float scale, const float* z, int lane,
                                             int32_t* __restrict__ topk,
                                             float* __restrict__ gates, float* __restrict__ probs, float (&my_g)[2],
                                             float (&my_p)[2]) {
  constexpr unsigned kAll = 0xffffffffu;
  const bool have[2] = {lane < E, lane + 32 < E};
  const float zv[2] = {have[0] ? z[lane] : 0.f, have[1] ? z[lane + 32] : 0.f};
  int slot[2] = {-1, -1};          // the slot in which this lane's expert was selected
  int sel[2] = {0, 0};             // lane j keeps the expert of slots j and j + 32
  int first = 0;
  float zmax = 0.f;
  for (int j = 0; j < k; ++j) {
    // this lane's candidate: its lower expert wins a tie ('>' is strict)
    int bi = -1;
    float bv = 0.f;
#pragma unroll
    for (int h = 0; h < 2; ++h)
      if (have[h] && slot[h] < 0 && (bi < 0 || zv[h] > bv)) { bi = lane + 32 * h; bv = zv[h]; }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(kAll, bv, o);
      const int oi = __shfl_xor_sync(kAll, bi, o);
      if (oi >= 0 && (bi < 0 || ov > bv || (ov == bv && oi < bi))) { bi = oi; bv = ov; }
    }
    if (j == 0) { first = bi; zmax = bv; }
    if ((bi & 31) == lane) slot[bi >> 5] = j;
    if ((j & 31) == lane) sel[j >> 5] = bi;
  }
  float ex[2];
#pragma unroll
  for (int h = 0; h < 2; ++h) ex[h] = have[h] ? expf((zv[h] - zmax) * scale) : 0.f;
  float psum = 0.f;
  for (int e = 0; e < min(E, 32); ++e) psum += __shfl_sync(kAll, ex[0], e);
  for (int e = 32; e < E; ++e) psum += __shfl_sync(kAll, ex[1], e - 32);
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    my_p[h] = have[h] ? ex[h] / psum : 0.f;
    my_g[h] = 0.f;
  }
  if (routing == BTX_ROUTE_SWITCH) {
#pragma unroll
    for (int h = 0; h < 2; ++h)
      if (slot[h] == 0) {          // the lane that owns the arg-max: the gate is its full-softmax probability
        my_g[h] = ex[h] / psum;
        topk[t] = first;
        gates[t] = my_g[h];
      }
  } else {
    float gsum = 0.f;
    for (int j = 0; j < k; ++j) {
      const int s = __shfl_sync(kAll, sel[j >> 5], j & 31);
      const float e0 = __shfl_sync(kAll, ex[0], s & 31), e1 = __shfl_sync(kAll, ex[1], s & 31);
      gsum += s < 32 ? e0 : e1;
    }
#pragma unroll
    for (int h = 0; h < 2; ++h)
      if (slot[h] >= 0) {          // the lane that owns a selected expert writes that slot
        my_g[h] = ex[h] / gsum;
        topk[(size_t)t * k + slot[h]] = lane + 32 * h;
        gates[(size_t)t * k + slot[h]] = my_g[h];
      }
  }
#pragma unroll
  for (int h = 0; h < 2; ++h)
    if (have[h]) probs[(size_t)t * E + lane + 32 * h] = my_p[h];
  __syncwarp();
}

// The same selection for up to 32 / G tokens at once when the layer has at most G <= 16 experts: G lanes per
// token, lane (slot, e) = (lane / G, lane % G) owns expert e of token i0 + slot.  z: the warp's logits in shared
// memory, kMaxExperts floats per token; tokens i0 .. min(i0 + 32 / G, nt) - 1 of the group starting at global
// token t0 are routed, their (unperturbed) logits stored, the Sample Top-1 noise added before the selection.
// Arithmetic and results per token are those of route_select.  On return lane e < E (slot 0) has had the gates
// and probabilities of expert e over the routed tokens added to u_sum and p_sum.
template <int G>
__device__ __forceinline__ void route_select_group(int t0, int i0, int nt, int E, int k, int routing, float scale,
                                                   const float* __restrict__ noise, float (*z)[kMaxExperts], int lane,
                                                   float* __restrict__ logits, int32_t* __restrict__ topk,
                                                   float* __restrict__ gates, float* __restrict__ probs, float& u_sum,
                                                   float& p_sum) {
  constexpr unsigned kAll = 0xffffffffu;
  const int slot = lane / G, e = lane % G, i = i0 + slot;
  const bool have = i < nt && e < E;
  const size_t t = (size_t)t0 + i;
  float zv = 0.f;
  if (have) {
    zv = z[i][e];
    logits[t * E + e] = zv;                               // reported logits are unperturbed
    if (noise != nullptr) zv = zv + noise[t * E + e];     // one fp32 addition decides the expert
  }
  int my_slot = -1;                // the slot in which this lane's expert was selected
  int sel = 0;                     // lane j of a group keeps the expert of slot j
  float zmax = 0.f;
  for (int j = 0; j < k; ++j) {
    int bi = have && my_slot < 0 ? e : -1;
    float bv = zv;
#pragma unroll
    for (int o = G / 2; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(kAll, bv, o);
      const int oi = __shfl_xor_sync(kAll, bi, o);
      if (oi >= 0 && (bi < 0 || ov > bv || (ov == bv && oi < bi))) { bi = oi; bv = ov; }
    }
    if (j == 0) zmax = bv;
    if (bi == e && have) my_slot = j;
    if (j == e) sel = bi;
  }
  const float ex = have ? expf((zv - zmax) * scale) : 0.f;
  float psum = 0.f;
  for (int ee = 0; ee < E; ++ee) psum += __shfl_sync(kAll, ex, ee, G);
  const float my_p = have ? ex / psum : 0.f;
  float my_g = 0.f;
  if (routing == BTX_ROUTE_SWITCH) {
    if (my_slot == 0) {            // the lane that owns the arg-max: the gate is its full-softmax probability
      my_g = ex / psum;
      topk[t] = e;
      gates[t] = my_g;
    }
  } else {
    float gsum = 0.f;
    for (int j = 0; j < k; ++j) {
      const int sj = __shfl_sync(kAll, sel, j, G);
      gsum += __shfl_sync(kAll, ex, sj < 0 ? 0 : sj, G);
    }
    if (my_slot >= 0) {            // the lane that owns a selected expert writes that slot
      my_g = ex / gsum;
      topk[t * k + my_slot] = e;
      gates[t * k + my_slot] = my_g;
    }
  }
  if (have) probs[t * E + e] = my_p;
  // gates and probabilities of expert e over the tokens of this pass, gathered in the first group's lanes
  float gs = my_g, ps = my_p;
#pragma unroll
  for (int o = 16; o >= G; o >>= 1) {
    gs += __shfl_xor_sync(kAll, gs, o);
    ps += __shfl_xor_sync(kAll, ps, o);
  }
  if (lane < E) { u_sum += gs; p_sum += ps; }
  __syncwarp();
}

constexpr int kSmallThreads = 256;
constexpr int kSmallMaxR = 1024;

// Batch means u and p, the loss, and the permutation of a small batch (R <= 1024) by ONE group of THREADS
// threads of a block (thread index `tid`, `sync()` a barrier of exactly those threads), from the per-token
// routing results already in global memory.  Every sum runs in a fixed order, so the result does not
// depend on which block runs this or on how many threads it has.
template <int THREADS, typename Sync>
__device__ __forceinline__ void small_batch_finish(int tid, Sync sync, int Tn, int E, int k, float alpha, int mt_max,
                                                   int r_pad_max, int cap,
                                                   const int32_t* topk, const float* gates, const float* probs,
                                                   float* __restrict__ u, float* __restrict__ p,
                                                   double* __restrict__ up64, float* __restrict__ loss,
                                                   int32_t* __restrict__ counts, int32_t* __restrict__ offsets,
                                                   int32_t* __restrict__ pad_offsets, int32_t* __restrict__ tile_expert,
                                                   int32_t* __restrict__ perm, int32_t* __restrict__ inv_perm,
                                                   int32_t* __restrict__ rowmap, int32_t* __restrict__ flat2row) {
  constexpr int NW = THREADS / 32;
  __shared__ double su[kMaxExperts], sp[kMaxExperts];
  __shared__ int hist[kMaxExperts + 1], running[kMaxExperts + 1], soff[kMaxExperts + 1], spad[kMaxExperts + 1];
  __shared__ int wcnt[NW][kMaxExperts + 1];
  const int warp = tid >> 5, lane = tid & 31;
  const int R = Tn * k;
  // ---- last block: batch means, loss ----
  for (int e = warp; e < E; e += NW) {
    double du = 0.0, dp = 0.0;
    for (int tt = lane; tt < Tn; tt += 32) {
      dp += (double)__ldcg(probs + (size_t)tt * E + e);
      for (int sl = 0; sl < k; ++sl)
        if (__ldcg(topk + (size_t)tt * k + sl) == e) du += (double)__ldcg(gates + (size_t)tt * k + sl);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      du += __shfl_xor_sync(0xffffffffu, du, o);
      dp += __shfl_xor_sync(0xffffffffu, dp, o);
    }
    if (lane == 0) {
      du /= (double)Tn; dp /= (double)Tn;
      su[e] = du; sp[e] = dp; u[e] = (float)du; p[e] = (float)dp; up64[e] = du; up64[E + e] = dp;
    }
  }
  // ---- permutation: histogram, scan, stable scatter in rounds of one block ----
  if (tid <= kMaxExperts) hist[tid] = 0;
  for (int j = tid; j < r_pad_max; j += THREADS) rowmap[j] = -1;
  if (cap < R)
    for (int j = tid; j < R; j += THREADS) perm[j] = -1;
  sync();
  for (int i = tid; i < R; i += THREADS) atomicAdd(&hist[__ldcg(topk + i)], 1);
  sync();
  if (tid == 0) {
    double acc = 0.0;
    for (int q = 0; q < E; ++q) acc += su[q] * sp[q];
    loss[0] = (float)((double)alpha * (double)E * acc);
    int o = 0, po = 0;
    for (int q = 0; q < E; ++q) {
      const int c = min(hist[q], cap);
      counts[q] = c; offsets[q] = o; pad_offsets[q] = po; soff[q] = o; spad[q] = po; running[q] = 0;
      o += c;
      po += (c + kRowTile - 1) / kRowTile * kRowTile;
    }
    offsets[E] = o; pad_offsets[E] = po; soff[E] = o; spad[E] = po;
  }
  sync();
  for (int mt = tid; mt < mt_max; mt += THREADS) {
    const int row = mt * kRowTile;
    int ex = -1;
    for (int q = 0; q < E; ++q)
      if (row >= spad[q] && row < spad[q + 1]) ex = q;
    tile_expert[mt] = ex;
  }
  for (int r0 = 0; r0 < R; r0 += THREADS) {
    for (int j = tid; j < NW * (kMaxExperts + 1); j += THREADS) (&wcnt[0][0])[j] = 0;
    sync();
    const int i = r0 + tid;
    const int e = (i < R) ? __ldcg(topk + i) : E;       // E = dummy bucket for idle lanes
    const unsigned same = __match_any_sync(0xffffffffu, e);
    const int rank = __popc(same & ((1u << lane) - 1u));
    if (rank == 0) wcnt[warp][e] = __popc(same);
    sync();
    if (i < R) {
      int before = 0;
      for (int w = 0; w < warp; ++w) before += wcnt[w][e];
      const int within = running[e] + before + rank;
      if (within < cap) {
        const int r = soff[e] + within, rp = spad[e] + within;
        perm[r] = i; inv_perm[i] = r; rowmap[rp] = i; flat2row[i] = rp;
      } else {
        inv_perm[i] = -1; flat2row[i] = -1;
      }
    }
    sync();
    if (tid < E) {
      int sum = 0;
      for (int w = 0; w < NW; ++w) sum += wcnt[w][tid];
      running[tid] += sum;
    }
    sync();
  }
}


// Logits of one token by eight warps that share its row: warp w takes every eighth 16-byte vector,
// part[w][e] receives its share of <x_t, W_l[e]>; the caller adds the eight parts in warp order.
template <typename T>
__device__ __forceinline__ void token_logit_parts(const T* __restrict__ xr, const T* __restrict__ wr, int d, int E,
                                                  int warp, int lane, float (*part)[kMaxExperts]) {
  constexpr int NW = kSmallThreads / 32;
  constexpr int VN = Vec<T>::N;
  for (int eb = 0; eb < E; eb += 8) {
    float acc[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[j] = 0.f;
#pragma unroll 2
    for (int c = (warp * 32 + lane) * VN; c < d; c += NW * 32 * VN) {
      float xv[VN];
      Vec<T>::load(xr + c, xv);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        if (eb + j < E) {
          float wv[VN];
          Vec<T>::load(wr + (size_t)(eb + j) * d + c, wv);
#pragma unroll
          for (int v = 0; v < VN; ++v) acc[j] = fmaf(xv[v], wv[v], acc[j]);
        }
      }
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      float a = acc[j];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
      if (lane == 0 && eb + j < E) part[warp][eb + j] = a;
    }
  }
}

}  // namespace routedev
}  // namespace btx
