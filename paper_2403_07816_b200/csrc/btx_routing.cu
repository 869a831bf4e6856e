// Router, load-balancing loss, token permutation, row gather / combine and router backward.
// These are the bandwidth- and latency-bound steps around the expert GEMMs.
//
//   router      logits = W_l x (Section 3.2), top-k by repeated arg-max with ties to the lower
//               index, gate softmax over the selected logits, full softmax, partial sums for
//               the batch means u and p of Section 3.3
//   finalize    u, p, L_LB = alpha E sum_i u_i p_i
//   permutation histogram -> exclusive scan -> stable scatter of the R assignments into
//               (expert ascending, token ascending) order; expert segments padded to whole 256-row tiles
//   gather      rows of x (or dy) copied into the padded expert-sorted layout
//   combine     y_t = sum over slots of the gate-scaled expert rows
//   router bwd  d logits from d gates and the two L_LB terms; dW_l = dz^T x; dx += W_l^T dz
#include "btx_common.cuh"

namespace btx {

namespace {

constexpr int kRouterThreads = 256;
constexpr int kRouterWarps = kRouterThreads / 32;
constexpr int kPermThreads = 256;
constexpr int kPermChunk = 1024;      // assignments per block of the permutation kernels

template <typename T> struct Vec;     // 16-byte vectors of the element type
template <> struct Vec<float> {
  static constexpr int N = 4;
  static __device__ __forceinline__ void load(const float* p, float (&v)[4]) {
    float4 q = *reinterpret_cast<const float4*>(p);
    v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
  }
};
template <> struct Vec<__nv_bfloat16> {
  static constexpr int N = 8;
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

// ---------------------------------------------------------------------------------------------
// Router
// ---------------------------------------------------------------------------------------------
// Selection, gates and softmax for one token from the logits z[0..E) in shared memory (all lanes of
// the calling warp take part).  The experts are chosen on z as it stands; the softmaxes are those of
// z * scale (scale = 1 except for Sample Top-1, whose temperature must not touch the arg-max: a
// rounded product could merge two distinct perturbed logits into a tie).  On return lane l holds the
// dense gate and probability of experts l (index 0) and l + 32 (index 1).
__device__ __forceinline__ void route_select(int t, int E, int k, int routing, float scale, const float* z, int lane,
                                             int32_t* __restrict__ topk,
                                             float* __restrict__ gates, float* __restrict__ probs, float (&my_g)[2],
                                             float (&my_p)[2]) {
  unsigned long long taken = 0;
  int sel[kMaxExperts];
  int first = 0;
  // repeated arg-max: strict '>' keeps the lower index on ties
  for (int j = 0; j < k; ++j) {
    int best = -1;
    float zb = 0.f;
    for (int e = 0; e < E; ++e) {
      if ((taken >> e) & 1ull) continue;
      float ze = z[e];
      if (best < 0 || ze > zb) { best = e; zb = ze; }
    }
    taken |= 1ull << best;
    sel[j] = best;
    if (j == 0) first = best;
  }
  const float zmax = z[first];
  float psum = 0.f;
  for (int e = 0; e < E; ++e) psum += expf((z[e] - zmax) * scale);
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int e = lane + 32 * h;
    my_p[h] = (e < E) ? expf((z[e] - zmax) * scale) / psum : 0.f;
    my_g[h] = 0.f;
  }
  if (routing == BTX_ROUTE_SWITCH) {
    float g0 = expf((z[first] - zmax) * scale) / psum;
    if ((first & 31) == lane) my_g[first >> 5] = g0;
    if (lane == 0) { topk[t] = first; gates[t] = g0; }
  } else {
    float gsum = 0.f;
    for (int j = 0; j < k; ++j) gsum += expf((z[sel[j]] - zmax) * scale);
    for (int j = 0; j < k; ++j) {
      float gj = expf((z[sel[j]] - zmax) * scale) / gsum;
      if ((sel[j] & 31) == lane) my_g[sel[j] >> 5] = gj;
      if (lane == 0) { topk[(size_t)t * k + j] = sel[j]; gates[(size_t)t * k + j] = gj; }
    }
  }
#pragma unroll
  for (int h = 0; h < 2; ++h)
    if (lane + 32 * h < E) probs[(size_t)t * E + lane + 32 * h] = my_p[h];
  __syncwarp();
}

// Routing of one token by one warp: logits (or the given ones), top-k by repeated arg-max with
// ties to the lower index, gates, full softmax.  `z` is this warp's shared scratch of kMaxExperts
// floats.  On return lane l holds the dense gate and the probability of experts l and l + 32.
template <typename T>
__device__ __forceinline__ void route_token(int t, int d, int E, int k, int routing, const T* __restrict__ x,
                                            const T* __restrict__ wr, const float* __restrict__ bias,
                                            const float* __restrict__ given_logits,
                                            const float* __restrict__ noise, float inv_tau, float* z, int lane,
                                            float* __restrict__ logits, int32_t* __restrict__ topk,
                                            float* __restrict__ gates, float* __restrict__ probs, float (&my_g)[2],
                                            float (&my_p)[2]) {
  constexpr int VN = Vec<T>::N;
  if (given_logits != nullptr) {
    for (int e = lane; e < E; e += 32) z[e] = given_logits[(size_t)t * E + e] + (bias ? bias[e] : 0.f);
  } else {
    const T* xr = x + (size_t)t * d;
    for (int eb = 0; eb < E; eb += 8) {
      float acc[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[j] = 0.f;
#pragma unroll 2
      for (int c = lane * VN; c < d; c += 32 * VN) {
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
        if (lane == 0 && eb + j < E) z[eb + j] = a + (bias ? bias[eb + j] : 0.f);
      }
    }
  }
  __syncwarp();
  for (int e = lane; e < E; e += 32) {
    logits[(size_t)t * E + e] = z[e];                             // reported logits are unperturbed
    if (noise != nullptr) z[e] = z[e] + noise[(size_t)t * E + e]; // one fp32 addition decides the expert
  }
  __syncwarp();
  route_select(t, E, k, routing, noise != nullptr ? inv_tau : 1.0f, z, lane, topk, gates, probs, my_g, my_p);
}

template <typename T>
__global__ void __launch_bounds__(kRouterThreads, 4)      // at most 64 registers: the x stream needs the occupancy
router_kernel(int Tn, int d, int E, int k, int routing, const T* __restrict__ x, const T* __restrict__ wr,
              const float* __restrict__ bias, const float* __restrict__ given_logits,
              const float* __restrict__ noise, float inv_tau,
              float* __restrict__ logits, int32_t* __restrict__ topk, float* __restrict__ gates,
              float* __restrict__ probs, float* __restrict__ route_part) {
  __shared__ float zs[kRouterWarps][kMaxExperts];
  __shared__ float red[kRouterWarps][kMaxExperts][2];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float u_acc[2] = {0.f, 0.f}, p_acc[2] = {0.f, 0.f};   // lane l accumulates experts l and l + 32 over this warp's tokens
  for (int t = blockIdx.x * kRouterWarps + warp; t < Tn; t += gridDim.x * kRouterWarps) {
    float my_g[2], my_p[2];
    route_token<T>(t, d, E, k, routing, x, wr, bias, given_logits, noise, inv_tau, zs[warp], lane, logits, topk, gates,
                   probs, my_g, my_p);
#pragma unroll
    for (int h = 0; h < 2; ++h) { u_acc[h] += my_g[h]; p_acc[h] += my_p[h]; }
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
}

// One warp per (expert, u|p) pair: lanes sum strided block partials in double, then a fixed-order
// shuffle tree, so the result does not depend on scheduling.
__global__ void __launch_bounds__(256)
lb_finalize_kernel(int Tn, int E, int nblocks, float alpha, const float* __restrict__ route_part,
                   float* __restrict__ u, float* __restrict__ p, float* __restrict__ loss, double* __restrict__ up64) {
  __shared__ double su[kMaxExperts], sp[kMaxExperts];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int pair = warp; pair < 2 * E; pair += 8) {
    double s = 0.0;
    for (int b = lane; b < nblocks; b += 32) s += (double)route_part[(size_t)b * 2 * E + pair];
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

// ---------------------------------------------------------------------------------------------
// Permutation
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kPermThreads)
perm_count_kernel(int R, int E, int nblocks, const int32_t* __restrict__ topk, int32_t* __restrict__ perm_counts) {
  __shared__ int hist[kMaxExperts];
  if (threadIdx.x < kMaxExperts) hist[threadIdx.x] = 0;
  __syncthreads();
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
perm_scatter_kernel(int R, int E, int nblocks, int cap, const int32_t* __restrict__ topk,
                    const int32_t* __restrict__ perm_base,
                    const int32_t* __restrict__ offsets, const int32_t* __restrict__ pad_offsets,
                    int32_t* __restrict__ perm, int32_t* __restrict__ inv_perm, int32_t* __restrict__ rowmap,
                    int32_t* __restrict__ flat2row) {
  constexpr int NW = kPermThreads / 32;
  __shared__ int running[kMaxExperts + 1];
  __shared__ int wcnt[NW][kMaxExperts + 1];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x < E) running[threadIdx.x] = perm_base[threadIdx.x * nblocks + blockIdx.x];
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
constexpr int kSmallThreads = 256;
constexpr int kSmallMaxR = 1024;

// Batch means u and p, the loss, and the permutation of a small batch (R <= 1024) by ONE block of THREADS
// threads, from the per-token routing results already in global memory.  Every sum runs in a fixed
// order, so the result does not depend on which block runs this or on how many threads it has.
template <int THREADS>
__device__ __forceinline__ void small_batch_finish(int Tn, int E, int k, float alpha, int mt_max, int r_pad_max, int cap,
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
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
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
  if (threadIdx.x <= kMaxExperts) hist[threadIdx.x] = 0;
  for (int j = threadIdx.x; j < r_pad_max; j += THREADS) rowmap[j] = -1;
  if (cap < R)
    for (int j = threadIdx.x; j < R; j += THREADS) perm[j] = -1;
  __syncthreads();
  for (int i = threadIdx.x; i < R; i += THREADS) atomicAdd(&hist[__ldcg(topk + i)], 1);
  __syncthreads();
  if (threadIdx.x == 0) {
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
  __syncthreads();
  for (int mt = threadIdx.x; mt < mt_max; mt += THREADS) {
    const int row = mt * kRowTile;
    int ex = -1;
    for (int q = 0; q < E; ++q)
      if (row >= spad[q] && row < spad[q + 1]) ex = q;
    tile_expert[mt] = ex;
  }
  for (int r0 = 0; r0 < R; r0 += THREADS) {
    for (int j = threadIdx.x; j < NW * (kMaxExperts + 1); j += THREADS) (&wcnt[0][0])[j] = 0;
    __syncthreads();
    const int i = r0 + threadIdx.x;
    const int e = (i < R) ? __ldcg(topk + i) : E;       // E = dummy bucket for idle lanes
    const unsigned same = __match_any_sync(0xffffffffu, e);
    const int rank = __popc(same & ((1u << lane) - 1u));
    if (rank == 0) wcnt[warp][e] = __popc(same);
    __syncthreads();
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
    __syncthreads();
    if (threadIdx.x < E) {
      int sum = 0;
      for (int w = 0; w < NW; ++w) sum += wcnt[w][threadIdx.x];
      running[threadIdx.x] += sum;
    }
    __syncthreads();
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

  small_batch_finish<kSmallThreads>(Tn, E, k, alpha, mt_max, r_pad_max, cap, topk, gates, probs, u, p, up64, loss, counts,
                                    offsets, pad_offsets, tile_expert, perm, inv_perm, rowmap, flat2row);
}

// The same routing for a handful of tokens whose expert kernels do not wait for it (they multiply every
// expert's weights with all tokens and look the routing up in their epilogues): one cluster of eight
// blocks, each taking every eighth token with the arithmetic of the kernel above; after a cluster
// barrier the first block forms the batch means, the loss and the permutation.  No ticket is needed.
// The kernel is launched as a programmatic dependent of the first expert kernel, which lets it start only
// after everything earlier in the stream is complete; it runs beside that kernel (256 threads of at most
// 64 registers fit next to one of its blocks) and, its work done, stays parked until that kernel has
// completed, so that whoever waits for this kernel has waited for both.
constexpr int kRouteCluster = 8;

template <typename T>
__global__ void __cluster_dims__(kRouteCluster, 1, 1) __launch_bounds__(kSmallThreads, 4)
route_permute_cluster_kernel(int Tn, int d, int E, int k, int routing, float alpha, int mt_max, int r_pad_max, int cap,
                             const T* __restrict__ x, const T* __restrict__ wr, const float* __restrict__ bias,
                             const float* __restrict__ noise, float inv_tau, float* logits, int32_t* topk, float* gates,
                             float* probs, float* __restrict__ u, float* __restrict__ p, double* __restrict__ up64,
                             float* __restrict__ loss, int32_t* __restrict__ counts, int32_t* __restrict__ offsets,
                             int32_t* __restrict__ pad_offsets, int32_t* __restrict__ tile_expert,
                             int32_t* __restrict__ perm, int32_t* __restrict__ inv_perm, int32_t* __restrict__ rowmap,
                             int32_t* __restrict__ flat2row) {
  constexpr int NW = kSmallThreads / 32;
  __shared__ float part[NW][kMaxExperts];
  __shared__ float z[kMaxExperts];
  allow_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int t = blockIdx.x; t < Tn; t += kRouteCluster) {
    token_logit_parts<T>(x + (size_t)t * d, wr, d, E, warp, lane, part);
    __syncthreads();
    if (threadIdx.x < E) {
      float a = 0.f;
      for (int w = 0; w < NW; ++w) a += part[w][threadIdx.x];
      a += bias ? bias[threadIdx.x] : 0.f;
      logits[(size_t)t * E + threadIdx.x] = a;
      if (noise != nullptr) a = a + noise[(size_t)t * E + threadIdx.x];
      z[threadIdx.x] = a;
    }
    __syncthreads();
    if (warp == 0) {
      float my_g[2], my_p[2];
      route_select(t, E, k, routing, noise != nullptr ? inv_tau : 1.0f, z, lane, topk, gates, probs, my_g, my_p);
    }
    __syncthreads();
  }
  // every block's routing results are visible to the first block after the cluster barrier
  __threadfence();
  __syncthreads();
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
  if (blockIdx.x == 0)
    small_batch_finish<kSmallThreads>(Tn, E, k, alpha, mt_max, r_pad_max, cap, topk, gates, probs, u, p, up64, loss, counts,
                                      offsets, pad_offsets, tile_expert, perm, inv_perm, rowmap, flat2row);
  grid_dependency_wait();
}

// ---------------------------------------------------------------------------------------------
// Gather into the padded sorted layout, combine out of it
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
gather_rows_kernel(int k, int row_vecs, const uint4* __restrict__ src, uint4* __restrict__ dst,
                   const int32_t* __restrict__ rowmap, const int32_t* __restrict__ pad_offsets, int E) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  allow_dependents();
  grid_dependency_wait();
  const int total = pad_offsets[E];
  for (int rp = blockIdx.x * 8 + warp; rp < total; rp += gridDim.x * 8) {
    int flat = rowmap[rp];
    uint4* o = dst + (size_t)rp * row_vecs;
    if (flat < 0) {
      for (int c = lane; c < row_vecs; c += 32) o[c] = make_uint4(0, 0, 0, 0);
    } else {
      const uint4* s = src + (size_t)(flat / k) * row_vecs;
#pragma unroll 4
      for (int c = lane; c < row_vecs; c += 32) o[c] = s[c];
    }
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
// row was never written and counts as zero.
template <typename T>
__global__ void __launch_bounds__(256)
combine_kernel(int Tn, int d, int k, int E, int splits, const float* __restrict__ rows, const float* __restrict__ dz,
               const T* __restrict__ wr, const int32_t* __restrict__ kept, T* __restrict__ y) {
  const size_t split_stride = (size_t)Tn * k * d;
  const int vecs = d >> 2;
  allow_dependents();
  grid_dependency_wait();
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < (size_t)Tn * vecs;
       i += (size_t)gridDim.x * blockDim.x) {
    int t = (int)(i / vecs), c = (int)(i % vecs) * 4;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s = 0; s < k; ++s) {
      if (kept != nullptr && kept[(size_t)t * k + s] < 0) continue;
      for (int sp = 0; sp < splits; ++sp) {
        float4 v = *reinterpret_cast<const float4*>(rows + sp * split_stride + ((size_t)t * k + s) * d + c);
        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
      }
    }
    if (dz != nullptr) {
      for (int e = 0; e < E; ++e) {
        float g = dz[(size_t)t * E + e];
        const T* w = wr + (size_t)e * d + c;
        acc.x = fmaf(g, to_f32(w[0]), acc.x); acc.y = fmaf(g, to_f32(w[1]), acc.y);
        acc.z = fmaf(g, to_f32(w[2]), acc.z); acc.w = fmaf(g, to_f32(w[3]), acc.w);
      }
    }
    store4<T>(y + (size_t)t * d + c, acc);
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
cudaError_t launch_router(const Plan& pl, int dtype, int routing, float alpha, const void* x, const void* w_router,
                          const float* bias, const float* given_logits, const float* noise, float inv_tau,
                          const Buffers& b, cudaStream_t st) {
  if (dtype == BTX_BF16) {
    router_kernel<__nv_bfloat16><<<pl.route_blocks, kRouterThreads, 0, st>>>(
        pl.T, pl.d, pl.E, pl.k, routing, (const __nv_bfloat16*)x, (const __nv_bfloat16*)w_router, bias, given_logits,
        noise, inv_tau, b.logits, b.topk, b.gates, b.probs, b.route_part);
  } else {
    router_kernel<float><<<pl.route_blocks, kRouterThreads, 0, st>>>(
        pl.T, pl.d, pl.E, pl.k, routing, (const float*)x, (const float*)w_router, bias, given_logits, noise, inv_tau,
        b.logits, b.topk, b.gates, b.probs, b.route_part);
  }
  lb_finalize_kernel<<<1, 256, 0, st>>>(pl.T, pl.E, pl.route_blocks, alpha, b.route_part, b.u, b.p, b.loss, b.up64);
  return cudaGetLastError();
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

cudaError_t launch_route_permute_cluster(const Plan& pl, int routing, float alpha, const void* x, const void* w_router,
                                       const float* bias, const float* noise, float inv_tau, const Buffers& b,
                                       cudaStream_t st) {
  return launch_after_predecessor(route_permute_cluster_kernel<__nv_bfloat16>, dim3(kRouteCluster), dim3(kSmallThreads), 0, st, true,
                                  pl.T, pl.d, pl.E, pl.k, routing, alpha, pl.mt_max, pl.r_pad_max, pl.capacity,
                                  (const __nv_bfloat16*)x, (const __nv_bfloat16*)w_router, bias, noise, inv_tau, b.logits,
                                  b.topk, b.gates, b.probs, b.u, b.p, b.up64, b.loss, b.counts, b.offsets, b.pad_offsets,
                                  b.tile_expert, b.perm, b.inv_perm, b.rowmap, b.flat2row);
}

cudaError_t launch_permute(const Plan& pl, const Buffers& b, cudaStream_t st) {
  cudaError_t e = cudaMemsetAsync(b.rowmap, 0xFF, (size_t)pl.r_pad_max * sizeof(int32_t), st);
  if (e != cudaSuccess) return e;
  if (pl.capacity < pl.R) {      // the tail of perm past the kept rows reads -1
    e = cudaMemsetAsync(b.perm, 0xFF, (size_t)pl.R * sizeof(int32_t), st);
    if (e != cudaSuccess) return e;
  }
  perm_count_kernel<<<pl.perm_blocks, kPermThreads, 0, st>>>(pl.R, pl.E, pl.perm_blocks, b.topk, b.perm_counts);
  perm_scan_kernel<<<1, 256, 0, st>>>(pl.E, pl.perm_blocks, pl.mt_max, pl.capacity, b.perm_counts, b.perm_base, b.counts,
                                      b.offsets, b.pad_offsets, b.tile_expert);
  perm_scatter_kernel<<<pl.perm_blocks, kPermThreads, 0, st>>>(pl.R, pl.E, pl.perm_blocks, pl.capacity, b.topk, b.perm_base,
                                                               b.offsets, b.pad_offsets, b.perm, b.inv_perm, b.rowmap,
                                                               b.flat2row);
  return cudaGetLastError();
}

cudaError_t launch_gather_rows(const Plan& pl, const void* src, void* dst_sorted, const Buffers& b, cudaStream_t st) {
  int row_vecs = pl.d * pl.esize / 16;
  int blocks = min(pl.r_pad_max / 8, sm_count() * 16);
  // small batches: the gather's launch overlaps the routing kernel's run
  return launch_after_predecessor(gather_rows_kernel, dim3(blocks), dim3(256), 0, st, pl.small != 0, pl.k, row_vecs,
                                  (const uint4*)src, (uint4*)dst_sorted, (const int32_t*)b.rowmap,
                                  (const int32_t*)b.pad_offsets, pl.E);
}

cudaError_t launch_combine(const Plan& pl, int dtype, const float* rows, int splits, void* y, const Buffers& b,
                           cudaStream_t st) {
  size_t n = (size_t)pl.T * (pl.d / 4);
  int blocks = (int)min((n + 255) / 256, (size_t)sm_count() * 32);
  const int32_t* kept = pl.capped ? b.flat2row : nullptr;
  if (dtype == BTX_BF16)
    return launch_after_predecessor(combine_kernel<__nv_bfloat16>, dim3(blocks), dim3(256), 0, st, pl.small != 0, pl.T,
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
  size_t n = (size_t)pl.T * (pl.d / 4);
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
