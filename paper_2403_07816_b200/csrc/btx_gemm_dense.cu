// Forward of a handful of tokens (T <= 64, BF16, nothing kept for backward): the decode-shaped case.
//
// The layer is bound by reading every expert's weights once from HBM, and what is not streaming is
// waiting: for the routing, for the row gather, for kernel boundaries.  Here the expert kernels do not
// depend on the routing at all until their last step:
//
//   pass 1   act[e][t] = silu(W1_e x_t) * W3_e x_t   for EVERY expert e and ALL tokens t.  The weights
//            take the M side of the tensor-core tile and the T tokens (rounded up to 16) the N side, so
//            an MMA costs N/2 cycles and the extra (token, expert) pairs are free; x is read as it
//            stands, no gather.  A CTA stages 64 rows of W1 and the same 64 rows of W3 per stage: h1
//            sits in accumulator lanes 0..63 and h3 in lanes 64..127, the epilogue warps of the upper
//            lanes hand h3 to those of the lower lanes through shared memory, and the product is
//            written as bf16: no partial sums, no second kernel.
//   pass 2   rows[t*k+slot] = gate * W2_e act[e][t], written for the (token, expert) pairs the router
//            selected, found in its epilogue from topk.
//
// Launch order: pass 1, routing, pass 2, combine, each a programmatic dependent of the one before.  Pass 1
// sets up while the kernel before it still runs, waits for it (griddepcontrol.wait), and only then lets
// the routing kernel start: that one therefore finds the stream's earlier work complete, runs beside
// pass 1 on the registers and shared memory pass 1 leaves free, and stays parked on its own
// griddepcontrol.wait until pass 1 has completed, so that pass 2, which waits for the routing kernel,
// has waited for both.  (Measured: a TMA load that a dependent kernel issues before the kernel it
// depends on has completed is held back until then, so nothing is gained by loading early in a
// dependent; with the routing kernel first, pass 1 began to stream only when that kernel had exited.)
// Warp roles, barriers and bounded waits as in the other tensor-core kernels: warp 0 TMA producer,
// warp 1 MMA issuer (leader CTA of the pair), warps 2-9 epilogue.  The path is chosen on the host when
// every expert is expected to hold a token, so that streaming all of them wastes nothing.
#include <cmath>

#include "btx_tc_ptx.cuh"

namespace btx {
namespace {

using namespace tcx;

constexpr int XW = 128;                                  // weight rows per CTA and stage (256 per pair)
constexpr int XN_MAX = 64;                               // tokens at most (MMA N)
constexpr int XA_BYTES = XW * BK * 2;
constexpr int X_STAGES = 8;
constexpr int X_RING_BYTES = X_STAGES * (XA_BYTES + (XN_MAX / 2) * BK * 2);
constexpr int X_EPI_WARPS = 8;
constexpr int X_THREADS = 64 + X_EPI_WARPS * 32;
constexpr int X_CTL_BYTES = 256;
constexpr int X_XCHG_FLOATS = 2 * 32 * 64;               // [column half][column][row of the lower lanes]
constexpr int X_SMEM_BYTES = X_RING_BYTES + 1024 + X_CTL_BYTES + X_XCHG_FLOATS * 4;

struct DenseParams {
  int W;                        // weight rows per expert (F in pass 1, d in pass 2)
  int E, T, N, k, m_tiles, kb_total;
  const int32_t* topk;          // pass 2: routing results
  const int32_t* flat2row;
  const float* gates;
  __nv_bfloat16* act;           // [E][N][F]: pass 1 output, pass 2 token operand
  float* out;                   // pass 2: [T*k][d]
  int32_t* status;
};

__device__ __forceinline__ void mbar_arrive_release(uint32_t bar) {
  asm volatile("mbarrier.arrive.release.cta.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

template <int PASS>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(X_THREADS, 1)
tc_dense_kernel(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmA1,
                const __grid_constant__ CUtensorMap tmB, const DenseParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t ring = (raw + 1023u) & ~1023u;
  uint8_t* ctl = smem_raw + (ring - raw) + X_RING_BYTES;
  const uint32_t bar_full = smem_u32(ctl);                              // 8 x 8 B (used in the leader)
  const uint32_t bar_empty = bar_full + X_STAGES * 8;                   // 8 x 8 B
  const uint32_t bar_tfull = bar_empty + X_STAGES * 8;                  // 2 x 8 B
  const uint32_t bar_tempty = bar_tfull + 16;                           // 2 x 8 B (used in the leader)
  const uint32_t bar_xfull = bar_tempty + 16;                           // 4 x 8 B: h3 of a warp pair is in shared memory
  const uint32_t bar_xfree = bar_xfull + 32;                            // 4 x 8 B: ... and has been read
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ctl + 224);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ctl + 232);
  float* xchg = reinterpret_cast<float*>(ctl + X_CTL_BYTES);
  const uint32_t stage_bytes = XA_BYTES + (uint32_t)(p.N / 2) * (BK * 2);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  if (PASS == 2) allow_dependents();

  if (threadIdx.x == 0) {
    for (int s = 0; s < X_STAGES; ++s) { mbar_init(bar_full + s * 8, 1); mbar_init(bar_empty + s * 8, 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(bar_tfull + a * 8, 1); mbar_init(bar_tempty + a * 8, 2 * X_EPI_WARPS * 32); }
    for (int a = 0; a < 4; ++a) { mbar_init(bar_xfull + a * 8, 32); mbar_init(bar_xfree + a * 8, 32); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int n_total = p.E * p.m_tiles;                    // item = (expert, block of weight rows)
  // Everything above ran while the kernel before this one may still have been running.
  grid_dependency_wait();
  if (PASS == 1) {
    allow_dependents();                                   // the routing kernel may start: earlier work is complete
    if (blockIdx.x == 0 && threadIdx.x == 0) p.status[0] = 0;
  }

  if (warp == 0) {
    // ------------------------------- TMA producer (both CTAs) -------------------------------
    if (lane == 0) {
      uint32_t stage = 0, phase = 0;
      bool ok = true;
      for (int t = pair; t < n_total && ok; t += n_pairs) {
        const int e = t / p.m_tiles, mt = t - e * p.m_tiles;
        for (int kb = 0; kb < p.kb_total; ++kb) {
          if (!(ok = mbar_wait(bar_empty + stage * 8, phase ^ 1u, abort_flag, p.status))) break;
          const uint32_t full_local = bar_full + stage * 8;
          const uint32_t full = map_to_cta(full_local, 0);
          const uint32_t sA = ring + stage * stage_bytes, sB = sA + XA_BYTES;
          if (rank == 0) mbar_expect_tx(full_local, 2 * stage_bytes);
          if (PASS == 1) {
            const int row = mt * XW + (int)rank * 64;      // this CTA: 64 rows of W1 over the same 64 rows of W3
            tma_load_3d(sA, &tmA0, kb * BK, row, e, full);
            tma_load_3d(sA + 64 * BK * 2, &tmA1, kb * BK, row, e, full);
          } else {
            tma_load_3d(sA, &tmA0, kb * BK, mt * 2 * XW + (int)rank * XW, e, full);
          }
          // this CTA's half of the N token rows
          tma_load_2d(sB, &tmB, kb * BK, (PASS == 1 ? 0 : e * p.N) + (int)rank * (p.N / 2), full);
          if (++stage == X_STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      for (int i = 0; i < X_STAGES && ok; ++i) {          // drain: all commits to this CTA have landed
        ok = mbar_wait(bar_empty + stage * 8, phase ^ 1u, abort_flag, p.status);
        if (++stage == X_STAGES) { stage = 0; phase ^= 1u; }
      }
    }
  } else if (warp == 1) {
    // ------------------------------- MMA issuer (leader CTA only) -------------------------------
    if (lane == 0 && rank == 0) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.N >> 3) << 17) |
                             ((uint32_t)((2 * XW) >> 4) << 24);
      uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
      bool ok = true;
      for (int t = pair; t < n_total && ok; t += n_pairs) {
        if (!(ok = mbar_wait(bar_tempty + acc * 8, acc_phase ^ 1u, abort_flag, p.status))) break;
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + acc * 256;
        for (int kb = 0; kb < p.kb_total; ++kb) {
          if (!(ok = mbar_wait(bar_full + stage * 8, phase, abort_flag, p.status))) break;
          tc_fence_after();
          const uint32_t sA = ring + stage * stage_bytes, sB = sA + XA_BYTES;
          const uint64_t da = smem_desc(sA, false), db = smem_desc(sB, false);
#pragma unroll
          for (int k16 = 0; k16 < BK / 16; ++k16)
            tc_mma_pair(tmem_d, da + (uint64_t)(2 * k16), db + (uint64_t)(2 * k16), idesc, (kb > 0 || k16 > 0) ? 1u : 0u);
          tc_commit_pair(bar_empty + stage * 8);
          if (++stage == X_STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tc_commit_pair(bar_tfull + acc * 8);
        acc ^= 1u;
        if (acc == 0) acc_phase ^= 1u;
      }
    }
  } else {
    // ------------------------------- epilogue (both CTAs) -------------------------------
    const int q = warp & 3, half = (warp - 2) >> 2;       // TMEM lane quarter; which 32 of the (at most) 64 token columns
    const int c0 = half * 32;
    const bool active = c0 < p.N;
    const uint32_t tempty_leader = map_to_cta(bar_tempty, 0);
    const uint32_t xfull = bar_xfull + (uint32_t)(half * 2 + (q & 1)) * 8, xfree = bar_xfree + (uint32_t)(half * 2 + (q & 1)) * 8;
    float* xs = xchg + half * (32 * 64);
    uint32_t acc = 0, acc_phase = 0, xphase = 0;
    bool ok = true;
    for (int t = pair; t < n_total && ok; t += n_pairs) {
      const int e = t / p.m_tiles, mt = t - e * p.m_tiles;
      if (!(ok = mbar_wait(bar_tfull + acc * 8, acc_phase, abort_flag, p.status))) break;
      tc_fence_after();
      if (active) {
        float v[32];
        if (PASS == 1) {
          tc_ld32(tmem_base + acc * 256 + c0 + ((uint32_t)(q * 32) << 16), v);
          if (q >= 2) {                                   // h3 rows: hand them to the warp that holds h1 of the same rows
            if (!(ok = mbar_wait(xfree, xphase ^ 1u, abort_flag, p.status))) break;
#pragma unroll
            for (int i = 0; i < 32; ++i) xs[i * 64 + (q - 2) * 32 + lane] = v[i];
            mbar_arrive_release(xfull);
          } else {
            if (!(ok = mbar_wait(xfull, xphase, abort_flag, p.status))) break;
            float w[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) w[i] = xs[i * 64 + q * 32 + lane];
            mbar_arrive_release(xfree);
            const int f = mt * XW + (int)rank * 64 + q * 32 + lane;
            if (f < p.W) {
              __nv_bfloat16* o = p.act + (size_t)e * p.N * p.W + f;
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (c0 + i < p.T) o[(size_t)(c0 + i) * p.W] = __float2bfloat16_rn(fast_swiglu(v[i], w[i]));
            }
          }
          xphase ^= 1u;
        } else {
          // lane i looks up token column c0 + i: the slot in which that token selected this expert, if any
          const int tok = c0 + lane;
          int my_flat = -1;
          if (tok < p.T)
            for (int s = 0; s < p.k; ++s) {
              const int fl = tok * p.k + s;
              if (p.topk[fl] == e && p.flat2row[fl] >= 0) my_flat = fl;
            }
          const float my_gate = my_flat >= 0 ? p.gates[my_flat] : 0.f;
          tc_ld32(tmem_base + acc * 256 + c0 + ((uint32_t)(q * 32) << 16), v);
          const int wrow = mt * 2 * XW + (int)rank * XW + q * 32 + lane;
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const int flat = __shfl_sync(0xffffffffu, my_flat, i);
            const float g = __shfl_sync(0xffffffffu, my_gate, i);
            if (flat >= 0 && wrow < p.W) p.out[(size_t)flat * p.W + wrow] = g * v[i];   // a 128-byte line per warp
          }
        }
      }
      tc_fence_before();
      mbar_arrive_cluster(tempty_leader + acc * 8);
      acc ^= 1u;
      if (acc == 0) acc_phase ^= 1u;
    }
  }

  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512));
  }
}

template <int PASS>
btx_status launch_dense(const CUtensorMap& a0, const CUtensorMap& a1, const CUtensorMap& b, const DenseParams& p,
                        cudaStream_t st) {
  if (cudaFuncSetAttribute(tc_dense_kernel<PASS>, cudaFuncAttributeMaxDynamicSharedMemorySize, X_SMEM_BYTES) != cudaSuccess)
    return BTX_ERR_CUDA;
  int pairs = sm_count() / 2;
  if (pairs > p.E * p.m_tiles) pairs = p.E * p.m_tiles;
  if (pairs < 1) pairs = 1;
  return launch_after_predecessor(tc_dense_kernel<PASS>, dim3(2 * pairs), dim3(X_THREADS), X_SMEM_BYTES, st, true, a0, a1,
                                  b, p) == cudaSuccess ? BTX_OK : BTX_ERR_CUDA;
}

}  // namespace

// Chosen for BF16 forwards that keep nothing for backward, hold at most 64 tokens, and are expected to
// leave under 5 % of the expert weights without a token (uniform routing: (1 - k/E)^T).
bool dense_small_fits(const Plan& pl, int save_for_backward) {
  if (save_for_backward || pl.esize != 2 || pl.T > XN_MAX || pl.R > 1024) return false;
  return std::pow(1.0 - (double)pl.k / (double)pl.E, (double)pl.T) <= 0.05;
}

btx_status launch_expert_forward_dense_bf16(const Plan& pl, int routing, float alpha, const void* x, const void* w_router,
                                            const float* bias, const float* noise, float inv_tau, const void* w1,
                                            const void* w3, const void* w2, const Buffers& b, cudaStream_t st) {
  const uint64_t d = pl.d, F = pl.F, E = pl.E;
  const uint32_t N = (uint32_t)pl.dense_n;
  CUtensorMap m0, m1, mx;
  btx_status s;
  DenseParams p = {};
  p.E = pl.E; p.T = pl.T; p.N = pl.dense_n; p.k = pl.k; p.status = b.status;
  p.topk = b.topk; p.flat2row = b.flat2row; p.gates = b.gates;
  p.act = (__nv_bfloat16*)b.act; p.out = b.yp;
  // pass 1: act = SwiGLU(x W1^T, x W3^T), all experts, all tokens (clears the status word)
  if (!make_map(&m0, w1, d, F, E, 64, 64) || !make_map(&m1, w3, d, F, E, 64, 64) || !make_map(&mx, x, d, pl.T, 0, 64, N / 2))
    return BTX_ERR_CUDA;
  p.W = pl.F; p.m_tiles = (pl.F + XW - 1) / XW; p.kb_total = (pl.d + BK - 1) / BK;
  if ((s = launch_dense<1>(m0, m1, mx, p, st)) != BTX_OK) return s;
  // routing, beside pass 1
  if (launch_route_permute_cluster(pl, routing, alpha, x, w_router, bias, noise, inv_tau, b, st) != cudaSuccess)
    return BTX_ERR_CUDA;
  mark_stage(2, st);
  // pass 2: gate-scaled rows of the selected (token, expert) pairs
  if (!make_map(&m0, w2, F, d, E, 64, XW) || !make_map(&mx, b.act, F, E * N, 0, 64, N / 2)) return BTX_ERR_CUDA;
  p.W = pl.d; p.m_tiles = (pl.d + 2 * XW - 1) / (2 * XW); p.kb_total = (pl.F + BK - 1) / BK;
  return launch_dense<2>(m0, m0, mx, p, st);
}

}  // namespace btx
