// Forward of a handful of tokens (T <= 64, BF16, nothing kept for backward) as ONE kernel: the
// decode-shaped case.
//
// The layer is bound by reading every expert's weights once from HBM, and what is not streaming is
// waiting: for the routing, for the row gather, for kernel boundaries (a kernel that follows a
// weight-streaming kernel of 148 blocks starts 5-10 us after its last block has finished, even when it was
// launched early as a programmatic dependent; measured with %globaltimer stamps).  Here the whole layer is a
// cooperative launch of one CTA pair per two multiprocessors with two grid-wide barriers:
//
//   routing  the eight epilogue warps of block t route token t (logits, top-k, gates, softmax) while the
//            first weight tiles of pass 1 arrive; nothing below needs the result before pass 2's epilogue
//   pass 1   act[e][t] = silu(W1_e x_t) * W3_e x_t   for EVERY expert e and ALL tokens t.  The weights
//            take the M side of the tensor-core tile and the T tokens (rounded up to 16) the N side, so
//            an MMA costs N/2 cycles and the extra (token, expert) pairs are free; x is read as it
//            stands, no gather.  A CTA stages 64 rows of W1 and the same 64 rows of W3 per stage: h1
//            sits in accumulator lanes 0..63 and h3 in lanes 64..127, the epilogue warps of the upper
//            lanes hand h3 to those of the lower lanes through shared memory, and the product is
//            written as bf16: no partial sums
//   -------- grid barrier (the first K blocks of W2, which depend on nothing, enter the ring before it) --------
//   pass 2   rows[t*k+slot] = gate * W2_e act[e][t], written for the (token, expert) pairs the router
//            selected (and, under a capacity limit, kept), found in the epilogue from topk.  Meanwhile the
//            epilogue warps of block 0 form the batch means, the loss and the permutation
//   -------- grid barrier --------
//   combine  y[t] = sum over slots of rows[t*k+slot], rounded once
//
// Warp roles, barriers and bounded waits as in the other tensor-core kernels: warps 0, 10, 11 TMA producers, warp 1
// MMA issuer (leader CTA of the pair), warps 2-9 epilogue; the TMA ring, the two TMEM accumulators and
// their barrier phases simply carry on from pass 1 to pass 2.  Every thread reaches both grid barriers
// whatever happened before (a wait that ran out only makes its role skip the rest of its work).  The path
// is chosen on the host when every expert is expected to hold a token, so that streaming all of them
// wastes nothing.
#include <cooperative_groups.h>

#include <cmath>

#include "btx_route_dev.cuh"
#include "btx_tc_ptx.cuh"

namespace btx {
namespace {

using namespace tcx;
using namespace routedev;
namespace cg = cooperative_groups;

constexpr int XW = 128;                                  // weight rows per CTA and stage (256 per pair)
constexpr int XN_MAX = 64;                               // tokens at most (MMA N)
constexpr int XA_BYTES = XW * BK * 2;
constexpr int X_STAGES = 10;
constexpr int X_RING_BYTES = X_STAGES * (XA_BYTES + (XN_MAX / 2) * BK * 2);
constexpr int X_EPI_WARPS = 8;
constexpr int X_EPI_THREADS = X_EPI_WARPS * 32;
constexpr int X_THREADS = 64 + X_EPI_THREADS + 64;        // warps 10 and 11: two more TMA producers
constexpr int X_CTL_BYTES = 384;
constexpr int X_XCHG_FLOATS = 2 * 32 * 64;               // [column half][column][row of the lower lanes]
constexpr int X_SMEM_BYTES = X_RING_BYTES + 1024 + X_CTL_BYTES + X_XCHG_FLOATS * 4;
static_assert(16 * X_STAGES + 112 <= X_CTL_BYTES, "barriers and control words fit the control block");
static_assert(X_EPI_THREADS == kSmallThreads, "the epilogue warps run the routing code of a 256-thread block");

struct FusedParams {
  int d, F, E, T, N, k;         // N = T rounded up to a multiple of 16 (MMA N)
  int routing, cap, capped, mt_max, r_pad_max;
  float alpha, inv_tau;
  const __nv_bfloat16* x;
  const __nv_bfloat16* wr;
  const float* bias;
  const float* noise;
  float* logits; int32_t* topk; float* gates; float* probs;
  float* u; float* p; double* up64; float* loss;
  int32_t* counts; int32_t* offsets; int32_t* pad_offsets; int32_t* tile_expert;
  int32_t* perm; int32_t* inv_perm; int32_t* rowmap; int32_t* flat2row;
  __nv_bfloat16* act;           // [E][N][F]: pass 1 output, pass 2 token operand
  float* rows;                  // [T*k][d]: pass 2 output
  __nv_bfloat16* y;             // [T][d]
  int32_t* status;
};

__device__ __forceinline__ void mbar_arrive_release(uint32_t bar) {
  asm volatile("mbarrier.arrive.release.cta.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 1, %0;" ::"n"(X_EPI_THREADS) : "memory"); }
__device__ __forceinline__ void prefetch_map(const CUtensorMap* m) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(m) : "memory");
}

// Work split.  The weight rows of a pass, all experts one after the other, are counted in units of 16 rows
// and cut into chunks of `cap` units (one full tile of a CTA pair); chunk i goes to pair i mod n_pairs, so at
// any time the pairs read neighbouring chunks.  At the Llama-2-7B shape the last round of pass 1 then has a
// tile for 48 of the 74 pairs only; cutting what is left after the full rounds evenly among all pairs instead
// was measured 3-7 % slower (a tile with fewer rows takes about as long per K block as a full one), so the
// plain deal stayed.  A chunk that crosses the end of an expert is walked as two tiles.  The first half of a
// tile's capacity belongs to the pair's first CTA; a CTA fetches its units of a tile as boxes of 8, 4, 2 and 1
// units, a full share as one box on a path of its own (measured: every TMA operation the producer thread
// steps through, even one it skips under a predicate, costs it about 80 ns, and three skipped ones per K
// block took the stream from 5.7 to 4.3 TB/s).
constexpr int XU = 16;                                   // rows per unit
struct XTile { int e, u0, n; };                          // expert, first unit inside the expert, units of both CTAs
struct XWalk {                                           // a pair's walk over its chunks
  int next_chunk, stride, cap, upe, total;               // units per expert, units of all experts
  int cur, end;                                          // rest of the current chunk
};
__device__ __forceinline__ XWalk x_walk(int pair, int n_pairs, int E, int upe, int cap) {
  XWalk w;
  w.next_chunk = pair; w.stride = n_pairs; w.cap = cap; w.upe = upe; w.total = E * upe;
  w.cur = 0; w.end = 0;
  return w;
}
__device__ __forceinline__ bool x_next_tile(XWalk& w, XTile& tl) {
  if (w.cur >= w.end) {
    w.cur = w.next_chunk * w.cap;
    if (w.cur >= w.total) return false;
    w.end = min(w.total, w.cur + w.cap);
    w.next_chunk += w.stride;
  }
  tl.e = w.cur / w.upe;
  tl.u0 = w.cur - tl.e * w.upe;
  tl.n = min(w.end - w.cur, w.upe - tl.u0);
  w.cur += tl.n;
  return true;
}

// Tensor maps of the kernel: weights with boxes of 1, 2, 4 and 8 units of rows (index = log2 of the units).
struct XMaps {
  CUtensorMap w1[3], w3[3];      // 16, 32, 64 rows
  CUtensorMap w2[4];             // 16, 32, 64, 128 rows
  CUtensorMap x, act;            // the tokens: N/2 rows per box
};

// `mine` units of weight rows starting at `row` of expert e, K block kb, into shared memory at dst
template <int LG_MAX>
__device__ __forceinline__ void x_load_units(uint32_t dst, const CUtensorMap* maps, int mine, int kb, int row, int e,
                                             uint32_t bar) {
  int done = 0;
#pragma unroll
  for (int lg = LG_MAX; lg >= 0; --lg) {
    if (mine - done >= (1 << lg)) {
      tma_load_3d(dst + done * (XU * BK * 2), maps + lg, kb * BK, row + done * XU, e, bar);
      done += 1 << lg;
    }
  }
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(X_THREADS, 1)
tc_small_forward_kernel(const __grid_constant__ XMaps tm, const FusedParams p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ float rt_part[X_EPI_WARPS][kMaxExperts];     // routing scratch of the epilogue warps
  __shared__ float rt_z[kMaxExperts];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t ring = (raw + 1023u) & ~1023u;
  uint8_t* ctl = smem_raw + (ring - raw) + X_RING_BYTES;
  const uint32_t bar_full = smem_u32(ctl);                              // X_STAGES x 8 B (used in the leader)
  const uint32_t bar_empty = bar_full + X_STAGES * 8;                   // X_STAGES x 8 B
  const uint32_t bar_tfull = bar_empty + X_STAGES * 8;                  // 2 x 8 B
  const uint32_t bar_tempty = bar_tfull + 16;                           // 2 x 8 B (used in the leader)
  const uint32_t bar_xfull = bar_tempty + 16;                           // 4 x 8 B: h3 of a warp pair is in shared memory
  const uint32_t bar_xfree = bar_xfull + 32;                            // 4 x 8 B: ... and has been read
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ctl + 16 * X_STAGES + 96);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ctl + 16 * X_STAGES + 104);
  float* xchg = reinterpret_cast<float*>(ctl + X_CTL_BYTES);
  const uint32_t stage_bytes = XA_BYTES + (uint32_t)(p.N / 2) * (BK * 2);

  cg::grid_group grid = cg::this_grid();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < X_STAGES; ++s) { mbar_init(bar_full + s * 8, 1); mbar_init(bar_empty + s * 8, 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(bar_tfull + a * 8, 1); mbar_init(bar_tempty + a * 8, 2 * X_EPI_THREADS); }
    for (int a = 0; a < 4; ++a) { mbar_init(bar_xfull + a * 8, 32); mbar_init(bar_xfree + a * 8, 32); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if (blockIdx.x == 0) { p.status[0] = 0; p.status[1] = 0; }
    for (int i = 0; i < 3; ++i) { prefetch_map(&tm.w1[i]); prefetch_map(&tm.w3[i]); }
    for (int i = 0; i < 4; ++i) prefetch_map(&tm.w2[i]);
    prefetch_map(&tm.x); prefetch_map(&tm.act);
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

  // ---- routing: the epilogue warps of block t take token t (they have nothing else to do yet) ----
  if (warp >= 2 && warp < 2 + X_EPI_WARPS) {
    const int tid = threadIdx.x - 64, ew = tid >> 5;
    for (int t = blockIdx.x; t < p.T; t += gridDim.x) {
      token_logit_parts<__nv_bfloat16>(p.x + (size_t)t * p.d, p.wr, p.d, p.E, ew, lane, rt_part);
      epi_sync();
      if (tid < p.E) {
        float a = 0.f;
        for (int w = 0; w < X_EPI_WARPS; ++w) a += rt_part[w][tid];
        a += p.bias ? p.bias[tid] : 0.f;
        p.logits[(size_t)t * p.E + tid] = a;                          // reported logits are unperturbed
        if (p.noise != nullptr) a = a + p.noise[(size_t)t * p.E + tid];  // one fp32 addition decides the expert
        rt_z[tid] = a;
      }
      epi_sync();
      if (ew == 0) {
        float my_g[2], my_p[2];
        route_select(t, p.E, p.k, p.routing, p.noise != nullptr ? p.inv_tau : 1.0f, rt_z, lane, p.topk, p.gates, p.probs,
                     my_g, my_p);
      }
      epi_sync();
    }
  }

  // per-thread pipeline state of whichever role this thread has; it carries over from pass 1 to pass 2
  uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0, xphase = 0;
  int w2_ahead = 0;                      // K blocks of W2 that the first loader put into the ring before pass 2 began
  bool ok = true;

  // code left in status word 1 by the first wait that runs out: which wait, in which pass, in which block
#define SITE(n) ((n) | (pass << 4) | ((int)blockIdx.x << 8))
  for (int pass = 1; pass <= 2; ++pass) {
    const int W = pass == 1 ? p.F : p.d;                                 // weight rows per expert
    const int kb_total = pass == 1 ? (p.d + BK - 1) / BK : (p.F + BK - 1) / BK;
    const int upe = (W + XU - 1) / XU;                                   // units per expert
    const int hu = pass == 1 ? 4 : 8;                                    // units of a full tile per CTA: 64 (of W1 and of W3) or 128 rows
    XWalk walk = x_walk(pair, n_pairs, p.E, upe, 2 * hu);                // this pair's chunks of units
    XTile tl;

    const int prod = warp == 0 ? 0 : (warp == 2 + X_EPI_WARPS ? 1 : (warp == 3 + X_EPI_WARPS ? 2 : -1));
    if (prod >= 0) {
      // ------------------------------- TMA producers (both CTAs) -------------------------------
      // Three threads share the issue (every TMA operation costs its thread about 80 ns, a K block lasts
      // about 350): warp 0 arms the stage's barrier and loads W1 (pass 2: W2), warp 10 loads W3, warp 11 the
      // token tile; each waits for the stage to be free on its own.
      if (lane == 0 && !(prod == 1 && pass == 2)) {
        // K blocks [kb0, kb1) of tile t of pass ps
        auto load_tile = [&](int ps, const XTile& t, int kb0, int kb1) {
          const int thu = ps == 1 ? 4 : 8;
          const int mine = rank == 0 ? min(t.n, thu) : max(0, t.n - thu);   // this CTA's units of the tile
          const int row = (t.u0 + (int)rank * thu) * XU;
          const uint32_t tx = (uint32_t)t.n * (XU * BK * 2) * (ps == 1 ? 2u : 1u) + 2u * (stage_bytes - XA_BYTES);
          // A thread with nothing to load for this tile (the second CTA's weight loaders when the tile fits into
          // the first CTA's share) only counts the stages: the MMAs do not depend on it, so it must not wait
          // on barriers that may complete more than one phase ahead of it.
          const bool idle = prod != 2 && mine == 0;
          for (int kb = kb0; kb < kb1; ++kb) {
            if (idle) {
              if (++stage == X_STAGES) { stage = 0; phase ^= 1u; }
              continue;
            }
            if (!(ok = mbar_wait(bar_empty + stage * 8, phase ^ 1u, abort_flag, p.status, kWaitLimitNs,
                                 1 | (ps << 4) | ((int)blockIdx.x << 8))))
              break;
            const uint32_t full_local = bar_full + stage * 8;
            const uint32_t full = map_to_cta(full_local, 0);             // the leader collects both CTAs' bytes
            const uint32_t sA = ring + stage * stage_bytes, sB = sA + XA_BYTES;
            if (prod == 0) {
              if (rank == 0) mbar_expect_tx(full_local, tx);
              if (ps == 1) {                              // this CTA: up to 64 rows of W1 ...
                if (mine == thu) tma_load_3d(sA, &tm.w1[2], kb * BK, row, t.e, full);
                else x_load_units<2>(sA, tm.w1, mine, kb, row, t.e, full);
              } else {
                if (mine == thu) tma_load_3d(sA, &tm.w2[3], kb * BK, row, t.e, full);
                else x_load_units<3>(sA, tm.w2, mine, kb, row, t.e, full);
              }
            } else if (prod == 1) {                       // ... over the same rows of W3
              if (mine == thu) tma_load_3d(sA + 64 * BK * 2, &tm.w3[2], kb * BK, row, t.e, full);
              else x_load_units<2>(sA + 64 * BK * 2, tm.w3, mine, kb, row, t.e, full);
            } else {                                      // this CTA's half of the N token rows
              if (ps == 1) tma_load_2d(sB, &tm.x, kb * BK, (int)rank * (p.N / 2), full);
              else tma_load_2d(sB, &tm.act, kb * BK, t.e * p.N + (int)rank * (p.N / 2), full);
            }
            if (++stage == X_STAGES) { stage = 0; phase ^= 1u; }
          }
        };
        bool first = true;
        while (ok && x_next_tile(walk, tl)) {
          load_tile(pass, tl, (first && prod == 0) ? w2_ahead : 0, kb_total);
          first = false;
        }
        w2_ahead = 0;
        if (pass == 1 && prod == 0 && ok) {
          // W2 does not depend on pass 1: the first K blocks of this pair's first pass-2 tile enter the ring as
          // the last MMAs of pass 1 free its stages, ahead of the grid barrier; the stage barriers complete once
          // the act tiles, loaded after the barrier, have arrived as well.
          XWalk walk2 = x_walk(pair, n_pairs, p.E, (p.d + XU - 1) / XU, 16);
          XTile t2;
          if (x_next_tile(walk2, t2)) {
            w2_ahead = min(X_STAGES, (p.F + BK - 1) / BK);
            load_tile(2, t2, 0, w2_ahead);
          }
        }
        if (pass == 2 && prod == 0)
          for (int i = 0; i < X_STAGES && ok; ++i) {        // drain: all commits to this CTA have landed
            ok = mbar_wait(bar_empty + stage * 8, phase ^ 1u, abort_flag, p.status, kWaitLimitNs, SITE(7));
            if (++stage == X_STAGES) { stage = 0; phase ^= 1u; }
          }
      }
    } else if (warp == 1) {
      // ------------------------------- MMA issuer (leader CTA only) -------------------------------
      if (lane == 0 && rank == 0) {
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.N >> 3) << 17) |
                               ((uint32_t)((2 * XW) >> 4) << 24);
        while (ok && x_next_tile(walk, tl)) {
          if (!(ok = mbar_wait(bar_tempty + acc * 8, acc_phase ^ 1u, abort_flag, p.status, kWaitLimitNs, SITE(2)))) break;
          tc_fence_after();
          const uint32_t tmem_d = tmem_base + acc * 256;
          for (int kb = 0; kb < kb_total; ++kb) {
            if (!(ok = mbar_wait(bar_full + stage * 8, phase, abort_flag, p.status, kWaitLimitNs, SITE(3)))) break;
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
    } else if (warp < 2 + X_EPI_WARPS) {
      // ------------------------------- epilogue (both CTAs) -------------------------------
      const int q = warp & 3, half = (warp - 2) >> 2;     // TMEM lane quarter; which 32 of the (at most) 64 token columns
      const int c0 = half * 32;
      const bool active = c0 < p.N;
      const uint32_t tempty_leader = map_to_cta(bar_tempty, 0);
      const uint32_t xfull = bar_xfull + (uint32_t)(half * 2 + (q & 1)) * 8, xfree = bar_xfree + (uint32_t)(half * 2 + (q & 1)) * 8;
      float* xs = xchg + half * (32 * 64);
      if (pass == 2 && blockIdx.x == 0)                   // every block's routing results are visible since the barrier
        small_batch_finish<X_EPI_THREADS>((int)threadIdx.x - 64, [] { epi_sync(); }, p.T, p.E, p.k, p.alpha, p.mt_max,
                                          p.r_pad_max, p.cap, p.topk, p.gates, p.probs, p.u, p.p, p.up64, p.loss, p.counts,
                                          p.offsets, p.pad_offsets, p.tile_expert, p.perm, p.inv_perm, p.rowmap, p.flat2row);
      while (ok && x_next_tile(walk, tl)) {
        const int e = tl.e;
        const int mine = rank == 0 ? min(tl.n, hu) : max(0, tl.n - hu);
        const int row0 = (tl.u0 + (int)rank * hu) * XU;                 // first weight row of this CTA's part of the tile
        if (!(ok = mbar_wait(bar_tfull + acc * 8, acc_phase, abort_flag, p.status, kWaitLimitNs, SITE(4)))) break;
        tc_fence_after();
        if (active) {
          float v[32];
          if (pass == 1) {
            tc_ld32(tmem_base + acc * 256 + c0 + ((uint32_t)(q * 32) << 16), v);
            if (q >= 2) {                                 // h3 rows: hand them to the warp that holds h1 of the same rows
              if (!(ok = mbar_wait(xfree, xphase ^ 1u, abort_flag, p.status, kWaitLimitNs, SITE(5)))) break;
#pragma unroll
              for (int i = 0; i < 32; ++i) xs[i * 64 + (q - 2) * 32 + lane] = v[i];
              mbar_arrive_release(xfull);
            } else {
              if (!(ok = mbar_wait(xfull, xphase, abort_flag, p.status, kWaitLimitNs, SITE(6)))) break;
              float w[32];
#pragma unroll
              for (int i = 0; i < 32; ++i) w[i] = xs[i * 64 + q * 32 + lane];
              mbar_arrive_release(xfree);
              const int f = row0 + q * 32 + lane;
              if (q * 32 + lane < mine * XU && f < W) {
                __nv_bfloat16* o = p.act + (size_t)e * p.N * W + f;
#pragma unroll
                for (int i = 0; i < 32; ++i)
                  if (c0 + i < p.T) o[(size_t)(c0 + i) * W] = __float2bfloat16_rn(fast_swiglu(v[i], w[i]));
              }
            }
            xphase ^= 1u;
          } else {
            // lane i looks up token column c0 + i: the slot in which that token selected this expert, if any;
            // under a capacity limit the expert keeps its first `cap` tokens in token order
            const int tok = c0 + lane;
            int my_flat = -1;
            if (tok < p.T) {
              for (int s = 0; s < p.k; ++s)
                if (__ldcg(p.topk + tok * p.k + s) == e) my_flat = tok * p.k + s;
              if (my_flat >= 0 && p.capped) {
                int before = 0;
                for (int i = 0; i < tok * p.k; ++i) before += __ldcg(p.topk + i) == e ? 1 : 0;
                if (before >= p.cap) my_flat = -1;
              }
            }
            const float my_gate = my_flat >= 0 ? __ldcg(p.gates + my_flat) : 0.f;
            tc_ld32(tmem_base + acc * 256 + c0 + ((uint32_t)(q * 32) << 16), v);
            const int wrow = row0 + q * 32 + lane;
            const bool row_ok = q * 32 + lane < mine * XU && wrow < W;
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const int flat = __shfl_sync(0xffffffffu, my_flat, i);
              const float g = __shfl_sync(0xffffffffu, my_gate, i);
              if (flat >= 0 && row_ok) p.rows[(size_t)flat * W + wrow] = g * v[i];   // a 128-byte line per warp
            }
          }
        }
        tc_fence_before();
        mbar_arrive_cluster(tempty_leader + acc * 8);
        acc ^= 1u;
        if (acc == 0) acc_phase ^= 1u;
      }
    }

    // What this pass wrote with ordinary stores (act, the routing results, the expert rows) is read after the
    // barrier by other blocks, act by their TMA loads: order it for both kinds of access.
    asm volatile("fence.proxy.async.global;" ::: "memory");
    __threadfence();
    tc_fence_before();
    grid.sync();
    tc_fence_after();
    asm volatile("fence.proxy.async.global;" ::: "memory");
  }

#undef SITE
  // ---- combine: y[t] = sum over slots of the gate-scaled expert rows, 8 columns per thread ----
  {
    const int vecs = p.d >> 3;
    for (int i = blockIdx.x * X_THREADS + threadIdx.x; i < p.T * vecs; i += gridDim.x * X_THREADS) {
      const int t = i / vecs, c = (i - t * vecs) * 8;
      float4 a0 = make_float4(0.f, 0.f, 0.f, 0.f), a1 = a0;
      for (int s = 0; s < p.k; ++s) {
        if (p.capped && __ldcg(p.flat2row + t * p.k + s) < 0) continue;       // a dropped assignment: its row was never written
        const float* r = p.rows + ((size_t)t * p.k + s) * p.d + c;
        const float4 v0 = __ldcg(reinterpret_cast<const float4*>(r)), v1 = __ldcg(reinterpret_cast<const float4*>(r + 4));
        a0.x += v0.x; a0.y += v0.y; a0.z += v0.z; a0.w += v0.w;
        a1.x += v1.x; a1.y += v1.y; a1.z += v1.z; a1.w += v1.w;
      }
      const float f[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
      *reinterpret_cast<uint4*>(p.y + (size_t)t * p.d + c) = pack8(f);
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

}  // namespace

// Chosen for BF16 forwards that keep nothing for backward, hold at most 64 tokens, and are expected to
// leave under 5 % of the expert weights without a token (uniform routing: (1 - k/E)^T).
bool dense_small_fits(const Plan& pl, int save_for_backward) {
  if (save_for_backward || pl.esize != 2 || pl.T > XN_MAX || pl.R > 1024) return false;
  return std::pow(1.0 - (double)pl.k / (double)pl.E, (double)pl.T) <= 0.05;
}

btx_status launch_forward_small_fused_bf16(const Plan& pl, int routing, float alpha, const void* x, const void* w_router,
                                           const float* bias, const float* noise, float inv_tau, const void* w1,
                                           const void* w3, const void* w2, void* y, const Buffers& b, cudaStream_t st) {
  const uint64_t d = pl.d, F = pl.F, E = pl.E;
  const uint32_t N = (uint32_t)pl.dense_n;
  XMaps tm;
  for (int lg = 0; lg < 4; ++lg) {
    if (lg < 3 && (!make_map(&tm.w1[lg], w1, d, F, E, 64, XU << lg) || !make_map(&tm.w3[lg], w3, d, F, E, 64, XU << lg)))
      return BTX_ERR_CUDA;
    if (!make_map(&tm.w2[lg], w2, F, d, E, 64, XU << lg)) return BTX_ERR_CUDA;
  }
  if (!make_map(&tm.x, x, d, pl.T, 0, 64, N / 2) || !make_map(&tm.act, b.act, F, E * N, 0, 64, N / 2)) return BTX_ERR_CUDA;
  FusedParams p = {};
  p.d = pl.d; p.F = pl.F; p.E = pl.E; p.T = pl.T; p.N = pl.dense_n; p.k = pl.k;
  p.routing = routing; p.cap = pl.capacity; p.capped = pl.capped; p.mt_max = pl.mt_max; p.r_pad_max = pl.r_pad_max;
  p.alpha = alpha; p.inv_tau = inv_tau;
  p.x = (const __nv_bfloat16*)x; p.wr = (const __nv_bfloat16*)w_router; p.bias = bias; p.noise = noise;
  p.logits = b.logits; p.topk = b.topk; p.gates = b.gates; p.probs = b.probs;
  p.u = b.u; p.p = b.p; p.up64 = b.up64; p.loss = b.loss;
  p.counts = b.counts; p.offsets = b.offsets; p.pad_offsets = b.pad_offsets; p.tile_expert = b.tile_expert;
  p.perm = b.perm; p.inv_perm = b.inv_perm; p.rowmap = b.rowmap; p.flat2row = b.flat2row;
  p.act = (__nv_bfloat16*)b.act; p.rows = b.yp; p.y = (__nv_bfloat16*)y; p.status = b.status;
  if (cudaFuncSetAttribute(tc_small_forward_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, X_SMEM_BYTES) != cudaSuccess)
    return BTX_ERR_CUDA;
  int pairs = sm_count() / 2;
  if (pairs < 1) pairs = 1;
  // A cooperative launch: the grid barriers need every block resident, one per multiprocessor.
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs); cfg.blockDim = dim3(X_THREADS); cfg.dynamicSmemBytes = X_SMEM_BYTES; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;
  attr[0].val.cooperative = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, tc_small_forward_kernel, tm, p) == cudaSuccess ? BTX_OK : BTX_ERR_CUDA;
}

}  // namespace btx
