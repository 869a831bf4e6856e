// BF16 expert GEMMs on the 5th-generation tensor cores (tcgen05.mma, accumulators in TMEM,
// operands staged in shared memory by TMA), one persistent warp-specialised kernel template.
//
// Two CTAs on neighbouring SMs form a cluster and work on one 256 x 256 output tile with
// tcgen05.mma.cta_group::2: each CTA stages its own 128 rows of A and one half (128 of the 256
// columns) of B, so shared-memory fill and operand-read traffic per SM is two thirds of what a
// single-CTA 128 x 256 tile needs, and each CTA keeps a 128 x 256 fp32 accumulator in its TMEM.
//
//   warp 0      TMA producer (one lane): fills a 6-stage ring of (A 128x64, B 128x64) bf16 tiles;
//               both CTAs signal the leader CTA's "full" barrier.  The leader's producer also
//               draws the pair's next tile from a global counter and posts it to every role
//   warp 1      allocates TMEM; in the leader CTA one lane issues the MMAs for the pair and
//               commits (multicast) to the barriers of both CTAs
//   warps 2-9   epilogue: tcgen05.ld of the CTA's accumulator (one row per thread, two warps per
//               32-row TMEM quarter, each taking half of the columns), fused element-wise work,
//               32-byte-per-lane global stores.  Two accumulators (2 x 256 TMEM columns) let the
//               epilogue of tile i overlap the main loop of tile i+1.
//
// Modes (all grouped by expert through the 256-row padded sorted layout):
//   FWD1   [h1|h3] = Xs [W1;W3]^T, epilogue a = silu(h1)*h3        (Section 3.2, FF_i)
//   FWD2   rows   = a W2^T, epilogue gate scale + scatter to t*k+slot rows
//   DACT   dA'    = dYs W2, epilogue SwiGLU backward, g*a, row-dot <dA', a> (d gate)
//   DX     dXs    = dh1 W1 + dh3 W3 (contraction over 2F), epilogue scatter
//   WGRAD  dW_e   = P_e^T Q_e, contraction over the expert's token rows, fp32 output
// Operands whose contraction index is not contiguous in memory (weights in DACT/DX, both
// operands in WGRAD) are fed as MN-major shared-memory tiles, so nothing is ever transposed.
//
// Every mbarrier wait is bounded: after about two seconds it records BTX_ERR_TIMEOUT in the
// workspace status word, raises a CTA-wide abort flag and the kernel drains and returns.  Both
// CTAs always meet at a cluster barrier before they exit, so no remote arrival can target a CTA
// that has already left.
#include "btx_tc_ptx.cuh"

namespace btx {
namespace {

using namespace tcx;

constexpr int BM = 128;                                  // rows per CTA; the pair covers 2*BM = kRowTile
constexpr int BN = 256, STAGES = 6;
constexpr int A_BYTES = BM * BK * 2, B_BYTES = (BN / 2) * BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int EPI_WARPS = 8;
constexpr int TC_THREADS = 64 + EPI_WARPS * 32;
constexpr int SCHED_SLOTS = 4;                           // tile numbers in flight between the scheduler and its readers
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 + 256;
static_assert(STAGES * 16 + 48 + SCHED_SLOTS * 20 <= 256, "control block fits behind the ring");
constexpr int GROUP_N = 8;                               // column tiles per raster group
static_assert(2 * BM == kRowTile, "a CTA pair covers one padded row tile");

enum TcMode { G_FWD1 = 0, G_FWD2 = 1, G_DACT = 2, G_DX = 3, G_WGRAD = 4 };

struct TcParams {
  int d, F, E, r_pad_max;
  int n_tiles;                  // column tiles
  int m_tiles;                  // WGRAD: 256-row tiles per expert
  int kb_total;                 // K blocks per tile (grouped modes)
  int kb_half;                  // DX: K blocks of the first operand pair
  int M, N;                     // WGRAD: gradient columns (lane side) and rows; other modes: N = output columns
  const int32_t* tile_expert;
  const int32_t* pad_offsets;
  const int32_t* rowmap;
  const float* gates;
  const __nv_bfloat16* h1;
  const __nv_bfloat16* h3;
  __nv_bfloat16* o0;
  __nv_bfloat16* o1;
  __nv_bfloat16* o2;
  float* of;
  float* dg_part;
  int save, accumulate;
  int a_one, b_one;             // the MN-major A / B tile of a stage is one TMA box (chunked tensor map)
  int wide;                     // all epilogue rows start on 32-byte boundaries
  int32_t* status;
  int32_t* next_tile;           // tile counter of this launch (zero when the kernel starts)
};

// ---------------------------------------------------------------------------------------------
// Tile schedule.  A tile is 256 output rows (128 per CTA) by 256 columns; tiles are numbered in
// raster order (get_tile).  CTA pairs draw tile numbers from one global counter, so the tiles in
// flight are always a contiguous window of the raster, whose operand panels fit in L2, however the
// pairs' speeds differ.  The leader's producer thread draws the number and posts it to both CTAs
// (TileFeed); the other producer, the MMA issuer and the epilogue warps read it from there.
// ---------------------------------------------------------------------------------------------
struct Tile {
  int m0;        // first output row of the pair's tile
  int nt;        // column tile index
  int e;         // expert
  int k_base;    // WGRAD: first contraction row
  int kb;        // K blocks
};

struct TileFeed {
  uint32_t full, empty, slots;     // shared-memory addresses: SCHED_SLOTS barriers, barriers, words
  uint32_t empty_leader;           // `empty` in the leader CTA (shared::cluster address)
  uint32_t q, phase;
  volatile int* abort_flag;
  int32_t* status;

  __device__ __forceinline__ void init(uint32_t ctl_addr, volatile int* af, int32_t* st) {
    full = ctl_addr; empty = full + SCHED_SLOTS * 8; slots = empty + SCHED_SLOTS * 8;
    empty_leader = map_to_cta(empty, 0);
    q = 0; phase = 0; abort_flag = af; status = st;
  }
  __device__ __forceinline__ void advance() { if (++q == SCHED_SLOTS) { q = 0; phase ^= 1u; } }
  // Scheduler (one thread of the leader): next tile number, posted to both CTAs.  -1 on time-out.
  __device__ __forceinline__ int draw(int32_t* counter) {
    if (!mbar_wait(empty + q * 8, phase ^ 1u, abort_flag, status)) return -1;
    const int t = atomicAdd(counter, 1);
    post_word(slots + q * 4, full + q * 8, 0, (uint32_t)t);
    post_word(slots + q * 4, full + q * 8, 1, (uint32_t)t);
    advance();
    return t;
  }
  // Reader: the next posted tile number.  Called by one thread (whole_warp = false) or by all 32
  // lanes of a warp; one arrival per caller group hands the slot back.  -1 on time-out.
  __device__ __forceinline__ int next(bool whole_warp, bool releaser) {
    if (!mbar_wait(full + q * 8, phase, abort_flag, status)) return -1;
    const int t = (int)ld_shared_u32(slots + q * 4);
    if (whole_warp) __syncwarp();
    if (releaser) mbar_arrive_cluster(empty_leader + q * 8);
    advance();
    return t;
  }
};
// readers per slot: the peer's producer, the leader's MMA issuer, the epilogue warps of both CTAs
constexpr int SCHED_READERS = 2 + 2 * EPI_WARPS;

template <int MODE>
__device__ __forceinline__ int total_tiles(const TcParams& p) {
  if (MODE == G_WGRAD) return p.E * p.m_tiles * p.n_tiles;
  return (p.pad_offsets[p.E] / kRowTile) * p.n_tiles;
}

template <int MODE>
__device__ __forceinline__ Tile get_tile(const TcParams& p, int t) {
  Tile tl;
  int mt_count, local = t;
  if (MODE == G_WGRAD) {
    mt_count = p.m_tiles;
    tl.e = t / (p.m_tiles * p.n_tiles);
    local = t - tl.e * p.m_tiles * p.n_tiles;
  } else {
    mt_count = p.pad_offsets[p.E] / kRowTile;
  }
  // raster: groups of GROUP_N column tiles; inside a group rows advance slowest
  const int full = p.n_tiles / GROUP_N;
  const int in_full = full * mt_count * GROUP_N;
  int g, width, rem;
  if (local < in_full) { g = local / (mt_count * GROUP_N); rem = local - g * mt_count * GROUP_N; width = GROUP_N; }
  else { g = full; rem = local - in_full; width = p.n_tiles - full * GROUP_N; }
  const int mt = rem / width;
  tl.nt = g * GROUP_N + rem - mt * width;
  tl.m0 = mt * kRowTile;
  if (MODE == G_WGRAD) {
    tl.k_base = p.pad_offsets[tl.e];
    tl.kb = (p.pad_offsets[tl.e + 1] - tl.k_base) / BK;
  } else {
    tl.e = p.tile_expert[mt];
    tl.k_base = 0;
    tl.kb = p.kb_total;
  }
  return tl;
}

// ---------------------------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------------------------
template <int MODE>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(TC_THREADS, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmA1,
               const __grid_constant__ CUtensorMap tmB0, const __grid_constant__ CUtensorMap tmB1,
               const TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;                        // 1024-byte aligned ring
  uint8_t* ctl = smem_raw + (tiles - raw) + STAGES * STAGE_BYTES;       // barriers behind the ring
  const uint32_t bar_full = smem_u32(ctl);                              // STAGES x 8 B (used in the leader)
  const uint32_t bar_empty = bar_full + STAGES * 8;                     // STAGES x 8 B (each CTA its own)
  const uint32_t bar_tfull = bar_empty + STAGES * 8;                    // 2 x 8 B (each CTA its own)
  const uint32_t bar_tempty = bar_tfull + 16;                           // 2 x 8 B (used in the leader)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ctl + STAGES * 16 + 32);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ctl + STAGES * 16 + 40);
  TileFeed feed;
  feed.init(bar_full + STAGES * 16 + 48, abort_flag, p.status);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();                              // 0 = leader of the pair
  constexpr bool A_MN = (MODE == G_WGRAD);
  constexpr bool B_MN = (MODE == G_DACT || MODE == G_DX || MODE == G_WGRAD);

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(bar_full + s * 8, 1); mbar_init(bar_empty + s * 8, 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(bar_tfull + a * 8, 1); mbar_init(bar_tempty + a * 8, 2 * EPI_WARPS * 32); }
    for (int s = 0; s < SCHED_SLOTS; ++s) { mbar_init(feed.full + s * 8, 1); mbar_init(feed.empty + s * 8, SCHED_READERS); }
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
  cluster_sync_all();                                     // the peer's barriers exist before anyone signals them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // Launched as a programmatic dependent: everything above ran while the kernel before this one may still have
  // been running; nothing below (which reads what that kernel wrote) starts before it has completed.
  allow_dependents();
  grid_dependency_wait();
  const int n_total = total_tiles<MODE>(p);

  if (warp == 0) {
    // ------------------------------- TMA producer (both CTAs) -------------------------------
    if (lane == 0) {
      uint32_t stage = 0, phase = 0;
      uint32_t uses = 0;                                  // stages filled so far (for the final drain)
      bool ok = true;
      while (ok) {
        const int t = rank == 0 ? feed.draw(p.next_tile) : feed.next(false, true);
        if (t < 0 || t >= n_total) break;                 // timed out, or the raster is exhausted
        const Tile tl = get_tile<MODE>(p, t);
        const int m0 = tl.m0 + (int)rank * BM;            // this CTA's rows
        for (int kb = 0; kb < tl.kb; ++kb) {
          if (!(ok = mbar_wait(bar_empty + stage * 8, phase ^ 1u, abort_flag, p.status))) break;
          const uint32_t full_local = bar_full + stage * 8;
          const uint32_t full = map_to_cta(full_local, 0);                 // the leader collects both CTAs' bytes
          const uint32_t sA = tiles + stage * STAGE_BYTES, sB = sA + A_BYTES;
          if (rank == 0) mbar_expect_tx(full_local, 2 * STAGE_BYTES);
          if (MODE == G_FWD1) {
            // B tile = [128 rows of W1 | 128 rows of W3]: the leader stages W1, its peer W3
            tma_load_2d(sA, &tmA0, kb * BK, m0, full);
            tma_load_3d(sB, rank == 0 ? &tmB0 : &tmB1, kb * BK, tl.nt * 128, tl.e, full);
          } else if (MODE == G_FWD2) {
            tma_load_2d(sA, &tmA0, kb * BK, m0, full);
            tma_load_3d(sB, &tmB0, kb * BK, tl.nt * BN + (int)rank * 128, tl.e, full);
          } else if (MODE == G_DACT) {
            tma_load_2d(sA, &tmA0, kb * BK, m0, full);
            if (p.b_one) {
              tma_load_4d(sB, &tmB0, 0, kb * BK, tl.nt * (BN / 64) + (int)rank * 2, tl.e, full);
            } else {
#pragma unroll
              for (int j = 0; j < 2; ++j)
                tma_load_3d(sB + j * CHUNK_BYTES, &tmB0, tl.nt * BN + ((int)rank * 2 + j) * 64, kb * BK, tl.e, full);
            }
          } else if (MODE == G_DX) {
            const bool second = kb >= p.kb_half;
            const int kk = (second ? kb - p.kb_half : kb) * BK;
            tma_load_2d(sA, second ? &tmA1 : &tmA0, kk, m0, full);
            if (p.b_one) {
              tma_load_4d(sB, second ? &tmB1 : &tmB0, 0, kk, tl.nt * (BN / 64) + (int)rank * 2, tl.e, full);
            } else {
#pragma unroll
              for (int j = 0; j < 2; ++j)
                tma_load_3d(sB + j * CHUNK_BYTES, second ? &tmB1 : &tmB0, tl.nt * BN + ((int)rank * 2 + j) * 64, kk, tl.e,
                            full);
            }
          } else {
            const int row = tl.k_base + kb * BK;
            if (p.a_one) {
              tma_load_3d(sA, &tmA0, 0, row, m0 / 64, full);
            } else {
#pragma unroll
              for (int j = 0; j < 2; ++j) tma_load_2d(sA + j * CHUNK_BYTES, &tmA0, m0 + j * 64, row, full);
            }
            if (p.b_one) {
              tma_load_3d(sB, &tmB0, 0, row, tl.nt * (BN / 64) + (int)rank * 2, full);
            } else {
#pragma unroll
              for (int j = 0; j < 2; ++j)
                tma_load_2d(sB + j * CHUNK_BYTES, &tmB0, tl.nt * BN + ((int)rank * 2 + j) * 64, row, full);
            }
          }
          ++uses;
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      // Drain: wait until the MMAs that read this CTA's last stages have retired, i.e. until every
      // commit addressed to this CTA's "empty" barriers has landed.
      // (a slot that was never filled passes at once)
      (void)uses;
      for (int i = 0; i < STAGES && ok; ++i) {
        ok = mbar_wait(bar_empty + stage * 8, phase ^ 1u, abort_flag, p.status);
        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
      }
    }
  } else if (warp == 1) {
    // ------------------------------- MMA issuer (leader CTA only) -------------------------------
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((A_MN ? 1u : 0u) << 15) |
                                 ((B_MN ? 1u : 0u) << 16) | ((uint32_t)(BN >> 3) << 17) |
                                 ((uint32_t)((2 * BM) >> 4) << 24);
      uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
      bool ok = true;
      while (ok) {
        const int t = feed.next(false, true);
        if (t < 0 || t >= n_total) break;
        const Tile tl = get_tile<MODE>(p, t);
        if (tl.kb == 0) continue;
        if (!(ok = mbar_wait(bar_tempty + acc * 8, acc_phase ^ 1u, abort_flag, p.status))) break;
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + acc * BN;
        for (int kb = 0; kb < tl.kb; ++kb) {
          if (!(ok = mbar_wait(bar_full + stage * 8, phase, abort_flag, p.status))) break;
          tc_fence_after();
          const uint32_t sA = tiles + stage * STAGE_BYTES, sB = sA + A_BYTES;
          const uint64_t da = smem_desc(sA, A_MN), db = smem_desc(sB, B_MN);
#pragma unroll
          for (int k16 = 0; k16 < BK / 16; ++k16) {
            // advance 16 contraction elements: 32 B inside a K-major row, 16 rows (2048 B) MN-major
            const uint64_t ao = (uint64_t)((A_MN ? 2048 : 32) * k16 >> 4);
            const uint64_t bo = (uint64_t)((B_MN ? 2048 : 32) * k16 >> 4);
            tc_mma_pair(tmem_d, da + ao, db + bo, idesc, (kb > 0 || k16 > 0) ? 1u : 0u);
          }
          tc_commit_pair(bar_empty + stage * 8);         // frees the stage in both CTAs when these MMAs retire
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tc_commit_pair(bar_tfull + acc * 8);
        acc ^= 1u;
        if (acc == 0) acc_phase ^= 1u;
      }
    }
  } else {
    // ------------------------------- epilogue (both CTAs) -------------------------------
    const int q = warp & 3;                               // TMEM lane quarter this warp may read
    const int half = (warp - 2) >> 2;                     // which half of the accumulator columns
    const int row = q * 32 + lane;
    const bool wide = p.wide != 0;                        // 32-byte accesses allowed for this launch
    const uint32_t tempty_leader = map_to_cta(bar_tempty, 0);
    uint32_t acc = 0, acc_phase = 0;
    bool ok = true;
    while (ok) {
      const int t = feed.next(true, lane == 0);
      if (t < 0 || t >= n_total) break;
      const Tile tl = get_tile<MODE>(p, t);
      const bool have_acc = tl.kb > 0;
      if (have_acc) {
        if (!(ok = mbar_wait(bar_tfull + acc * 8, acc_phase, abort_flag, p.status))) break;
        tc_fence_after();
      }
      const uint32_t taddr = tmem_base + acc * BN + ((uint32_t)(q * 32) << 16);
      const int rp = tl.m0 + (int)rank * BM + row;
      float v[32];

      if (MODE == G_FWD1) {
        float w[32];
        const int F = p.F;
        for (int c = half * 64; c < half * 64 + 64; c += 32) {
          tc_ld32(taddr + c, v);
          tc_ld32(taddr + 128 + c, w);
          const int col = tl.nt * 128 + c;
#pragma unroll
          for (int g16 = 0; g16 < 2; ++g16) {
            if (col + g16 * 16 < F) {
              float a16[16];
#pragma unroll
              for (int i = 0; i < 16; ++i) a16[i] = fast_swiglu(v[g16 * 16 + i], w[g16 * 16 + i]);
              const size_t o = (size_t)rp * F + col + g16 * 16;
              st32(p.o0 + o, pack8(a16), pack8(a16 + 8), wide, col + g16 * 16 + 8 < F);
              if (p.save) {
                st32(p.o1 + o, pack8(v + g16 * 16), pack8(v + g16 * 16 + 8), wide, col + g16 * 16 + 8 < F);
                st32(p.o2 + o, pack8(w + g16 * 16), pack8(w + g16 * 16 + 8), wide, col + g16 * 16 + 8 < F);
              }
            }
          }
        }
      } else if (MODE == G_FWD2 || MODE == G_DX) {
        const int flat = p.rowmap[rp];
        const float g = (MODE == G_FWD2 && flat >= 0) ? p.gates[flat] : 1.0f;
        const int N = p.N;
        for (int c = half * (BN / 2); c < (half + 1) * (BN / 2); c += 32) {
          tc_ld32(taddr + c, v);
          const int col = tl.nt * BN + c;
          if (flat >= 0) {
            float* o = p.of + (size_t)flat * N + col;
#pragma unroll
            for (int g8 = 0; g8 < 4; ++g8)
              if (col + g8 * 8 < N) {
                float t8[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) t8[i] = g * v[g8 * 8 + i];
                st32(o + g8 * 8, f4(t8), f4(t8 + 4), wide);
              }
          }
        }
      } else if (MODE == G_DACT) {
        const int flat = p.rowmap[rp];
        const float g = flat >= 0 ? p.gates[flat] : 0.f;
        const int F = p.F;
        float rowdot = 0.f;
        for (int c = half * (BN / 2); c < (half + 1) * (BN / 2); c += 32) {
          const int col = tl.nt * BN + c;
          uint4 q1[4], q3[4];
#pragma unroll
          for (int g16 = 0; g16 < 2; ++g16) {
            if (col + g16 * 16 < F) {
              const size_t o = (size_t)rp * F + col + g16 * 16;
              ld32(p.h1 + o, q1[2 * g16], q1[2 * g16 + 1], wide, col + g16 * 16 + 8 < F);
              ld32(p.h3 + o, q3[2 * g16], q3[2 * g16 + 1], wide, col + g16 * 16 + 8 < F);
            }
          }
          tc_ld32(taddr + c, v);
#pragma unroll
          for (int g16 = 0; g16 < 2; ++g16) {
            if (col + g16 * 16 < F) {
              const size_t o = (size_t)rp * F + col + g16 * 16;
              float h1[16], h3[16], d1[16], d3[16], ga[16];
              unpack8(q1[2 * g16], h1); unpack8(q1[2 * g16 + 1], h1 + 8);
              unpack8(q3[2 * g16], h3); unpack8(q3[2 * g16 + 1], h3 + 8);
#pragma unroll
              for (int i = 0; i < 16; ++i) {
                const float da = v[g16 * 16 + i];
                const float sg = fast_sigmoid(h1[i]);
                const float hs = h1[i] * sg;
                const float a = hs * h3[i];
                const float gda = g * da;
                d1[i] = gda * h3[i] * sg * (1.0f + h1[i] * (1.0f - sg));
                d3[i] = gda * hs;
                ga[i] = g * a;
                rowdot = fmaf(da, a, rowdot);
              }
              st32(p.o0 + o, pack8(d1), pack8(d1 + 8), wide, col + g16 * 16 + 8 < F);
              st32(p.o1 + o, pack8(d3), pack8(d3 + 8), wide, col + g16 * 16 + 8 < F);
              st32(p.o2 + o, pack8(ga), pack8(ga + 8), wide, col + g16 * 16 + 8 < F);
            }
          }
        }
        p.dg_part[(size_t)(tl.nt * 2 + half) * p.r_pad_max + rp] = rowdot;
      } else {  // WGRAD, stored transposed: lane = column of the gradient, TMEM column = its row
        const int ncols = p.M, nrows = p.N;                // memory shape of one expert's gradient: [nrows][ncols]
        const bool lane_ok = rp < ncols;
        for (int c = half * (BN / 2); c < (half + 1) * (BN / 2); c += 32) {
          const int r0 = tl.nt * BN + c;
          if (r0 >= nrows) break;
          if (have_acc) tc_ld32(taddr + c, v);
          else {
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = 0.f;
          }
          if (lane_ok) {
            float* o = p.of + ((size_t)tl.e * nrows + r0) * ncols + rp;
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              if (r0 + i < nrows) {                        // one 128-byte line per warp instruction
                float x = v[i];
                if (p.accumulate) x += o[(size_t)i * ncols];
                o[(size_t)i * ncols] = x;
              }
            }
          }
        }
      }
      if (have_acc) {
        tc_fence_before();
        mbar_arrive_cluster(tempty_leader + acc * 8);     // the leader's MMA issuer waits for both CTAs
        acc ^= 1u;
        if (acc == 0) acc_phase ^= 1u;
      }
    }
  }

  // Nobody leaves before both CTAs are done: remote arrivals and multicast commits must find
  // their target barriers alive.
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512));
  }
}

// ---------------------------------------------------------------------------------------------
// Host side: tensor maps and launches
// ---------------------------------------------------------------------------------------------

template <int MODE>
btx_status launch_tc(const CUtensorMap& a0, const CUtensorMap& a1, const CUtensorMap& b0, const CUtensorMap& b1,
                     const TcParams& params, int max_tiles, int launch_index, cudaStream_t st) {
  // every launch of one forward or backward call draws from its own counter in the status block,
  // which the call zeroed before its first kernel
  TcParams p = params;
  p.next_tile = params.status + kTileCounterWord + launch_index;
  if (cudaFuncSetAttribute(tc_gemm_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess)
    return BTX_ERR_CUDA;
  int pairs = sm_count() / 2;
  if (pairs > max_tiles) pairs = max_tiles;
  if (pairs < 1) pairs = 1;
  // cluster dims are compiled in
  return launch_after_predecessor(tc_gemm_kernel<MODE>, dim3(2 * pairs), dim3(TC_THREADS), SMEM_BYTES, st, true, a0, a1, b0,
                                  b1, p) == cudaSuccess ? BTX_OK : BTX_ERR_CUDA;
}

// One thread waits, with a 50 ms limit, on a barrier that nobody will ever arrive at.
__global__ void wait_expiry_kernel(int32_t* status) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (threadIdx.x == 0) mbar_wait(smem_u32(&bar), 0u, &abort_flag, status, 50000000ull);
}

TcParams base_params(const Plan& pl, const Buffers& b) {
  TcParams p = {};
  p.d = pl.d; p.F = pl.F; p.E = pl.E; p.r_pad_max = pl.r_pad_max;
  p.tile_expert = b.tile_expert; p.pad_offsets = b.pad_offsets; p.rowmap = b.rowmap; p.gates = b.gates;
  p.status = b.status;
  return p;
}

}  // namespace

cudaError_t launch_wait_expiry_selftest(int32_t* status, cudaStream_t st) {
  wait_expiry_kernel<<<1, 32, 0, st>>>(status);
  return cudaGetLastError();
}

btx_status launch_expert_forward_bf16(const Plan& pl, const void* w1, const void* w3, const void* w2,
                                      const Buffers& b, int save, cudaStream_t st) {
  const uint64_t d = pl.d, F = pl.F, E = pl.E, RP = pl.r_pad_max;
  CUtensorMap a, b0, b1;
  btx_status s;
  // GEMM-1: [h1|h3] = Xs [W1;W3]^T with the SwiGLU epilogue
  if (!make_map(&a, b.xs, d, RP, 0, 64, 128) || !make_map(&b0, w1, d, F, E, 64, 128) ||
      !make_map(&b1, w3, d, F, E, 64, 128))
    return BTX_ERR_CUDA;
  TcParams p = base_params(pl, b);
  p.n_tiles = (pl.F + 127) / 128; p.kb_total = (pl.d + BK - 1) / BK; p.N = pl.F;
  p.o0 = (__nv_bfloat16*)b.act; p.o1 = (__nv_bfloat16*)b.h1; p.o2 = (__nv_bfloat16*)b.h3; p.save = save;
  const bool f_pitch32 = pl.F % 16 == 0;                  // bf16 rows of F elements start on 32-byte boundaries
  p.wide = f_pitch32 && aligned32(b.act) && aligned32(b.h1) && aligned32(b.h3);
  if ((s = launch_tc<G_FWD1>(a, a, b0, b1, p, pl.mt_max * p.n_tiles, 0, st)) != BTX_OK) return s;
  mark_stage(2, st);
  // GEMM-2: gate-scaled expert rows = act W2^T
  if (!make_map(&a, b.act, F, RP, 0, 64, 128) || !make_map(&b0, w2, F, d, E, 64, 128)) return BTX_ERR_CUDA;
  p.n_tiles = (pl.d + BN - 1) / BN; p.kb_total = (pl.F + BK - 1) / BK; p.N = pl.d; p.of = b.yp;
  p.wide = aligned32(b.yp);                               // fp32 rows of d (a multiple of 8) elements
  return launch_tc<G_FWD2>(a, a, b0, b0, p, pl.mt_max * p.n_tiles, 1, st);
}

btx_status launch_expert_backward_bf16(const Plan& pl, const void* w1, const void* w3, const void* w2,
                                       const Buffers& b, float* dw1, float* dw3, float* dw2, int accumulate,
                                       int skip_wgrad, cudaEvent_t after_dx, cudaStream_t st) {
  const uint64_t d = pl.d, F = pl.F, E = pl.E, RP = pl.r_pad_max;
  CUtensorMap a0, a1, b0, b1;
  btx_status s;
  TcParams p = base_params(pl, b);
  // dgrad-2: dA' = dYs W2 (W2[d,F] read N-major), SwiGLU backward epilogue
  if (!make_map(&a0, b.dys, d, RP, 0, 64, 128)) return BTX_ERR_CUDA;
  p.b_one = make_map_mn(&b0, w2, F, d, E);
  if (!p.b_one && !make_map(&b0, w2, F, d, E, 64, 64)) return BTX_ERR_CUDA;
  p.n_tiles = (pl.F + BN - 1) / BN; p.kb_total = (pl.d + BK - 1) / BK; p.N = pl.F;
  p.h1 = (const __nv_bfloat16*)b.h1; p.h3 = (const __nv_bfloat16*)b.h3;
  p.o0 = (__nv_bfloat16*)b.dh1; p.o1 = (__nv_bfloat16*)b.dh3; p.o2 = (__nv_bfloat16*)b.ga; p.dg_part = b.dg_part;
  p.wide = pl.F % 16 == 0 && aligned32(b.h1) && aligned32(b.h3) && aligned32(b.dh1) && aligned32(b.dh3) && aligned32(b.ga);
  if ((s = launch_tc<G_DACT>(a0, a0, b0, b0, p, pl.mt_max * p.n_tiles, 0, st)) != BTX_OK) return s;
  mark_stage(2, st);
  // dgrad-1: dXs = dh1 W1 + dh3 W3 (weights read N-major), scatter to t*k+slot rows
  if (!make_map(&a0, b.dh1, F, RP, 0, 64, 128) || !make_map(&a1, b.dh3, F, RP, 0, 64, 128)) return BTX_ERR_CUDA;
  p.b_one = make_map_mn(&b0, w1, d, F, E) && make_map_mn(&b1, w3, d, F, E);
  if (!p.b_one && (!make_map(&b0, w1, d, F, E, 64, 64) || !make_map(&b1, w3, d, F, E, 64, 64))) return BTX_ERR_CUDA;
  p.n_tiles = (pl.d + BN - 1) / BN; p.kb_half = (pl.F + BK - 1) / BK; p.kb_total = 2 * p.kb_half; p.N = pl.d;
  p.of = b.dxp; p.wide = aligned32(b.dxp);
  if ((s = launch_tc<G_DX>(a0, a1, b0, b1, p, pl.mt_max * p.n_tiles, 1, st)) != BTX_OK) return s;
  mark_stage(3, st);
  if (after_dx != nullptr && cudaEventRecord(after_dx, st) != cudaSuccess) return BTX_ERR_CUDA;   // the router backward may start here
  if (skip_wgrad) return BTX_OK;
  // wgrads: contraction over the expert's padded token rows, both operands MN-major.  The operand
  // indexed by the gradient's contiguous (column) index goes on the M side, so that the 32 lanes of
  // an epilogue warp write 32 neighbouring columns of one gradient row.
  p.accumulate = accumulate;
  p.a_one = make_map_mn(&a0, b.ga, F, RP, 0);
  p.b_one = make_map_mn(&b0, b.dys, d, RP, 0);
  if ((!p.a_one && !make_map(&a0, b.ga, F, RP, 0, 64, 64)) || (!p.b_one && !make_map(&b0, b.dys, d, RP, 0, 64, 64)))
    return BTX_ERR_CUDA;
  p.M = pl.F; p.N = pl.d; p.m_tiles = (pl.F + kRowTile - 1) / kRowTile; p.n_tiles = (pl.d + BN - 1) / BN; p.of = dw2;
  if ((s = launch_tc<G_WGRAD>(a0, a0, b0, b0, p, pl.E * p.m_tiles * p.n_tiles, 2, st)) != BTX_OK) return s;
  mark_stage(4, st);
  p.a_one = make_map_mn(&a0, b.xs, d, RP, 0);
  p.b_one = make_map_mn(&b0, b.dh1, F, RP, 0) && make_map_mn(&b1, b.dh3, F, RP, 0);
  if ((!p.a_one && !make_map(&a0, b.xs, d, RP, 0, 64, 64)) ||
      (!p.b_one && (!make_map(&b0, b.dh1, F, RP, 0, 64, 64) || !make_map(&b1, b.dh3, F, RP, 0, 64, 64))))
    return BTX_ERR_CUDA;
  p.M = pl.d; p.N = pl.F; p.m_tiles = (pl.d + kRowTile - 1) / kRowTile; p.n_tiles = (pl.F + BN - 1) / BN; p.of = dw1;
  if ((s = launch_tc<G_WGRAD>(a0, a0, b0, b0, p, pl.E * p.m_tiles * p.n_tiles, 3, st)) != BTX_OK) return s;
  mark_stage(5, st);
  p.of = dw3;
  s = launch_tc<G_WGRAD>(a0, a0, b1, b1, p, pl.E * p.m_tiles * p.n_tiles, 4, st);
  mark_stage(6, st);
  return s;
}

}  // namespace btx
