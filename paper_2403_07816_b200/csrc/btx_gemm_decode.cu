// Weight-streaming expert GEMMs for small batches (T*k <= 1024, the decode-shaped case), BF16.
//
// With a few tokens per expert the layer is bound by reading the expert weights once from HBM.
// The weights therefore take the M side of the tensor-core tile (256 weight rows per CTA pair,
// tcgen05.mma.cta_group::2) and the tokens of one padded 256-row tile of an expert take the N side,
// N = the tile's real rows rounded up to 16: with 16 tokens an MMA costs 8 cycles instead of 128, so
// the tensor pipe does not limit the stream, and nothing is spent on padding rows.  The contraction is split
// into S parts per tile so that the number of work items is a multiple of the CTA pairs; every
// item writes its fp32 partial product for the valid tokens only, addressed [split][t*k+slot][row]:
// a lane owns a weight row, so the 32 lanes of a warp write one 128-byte line per token.
//
//   pass 1   partial h1, h3 = W1_e x, W3_e x   -> swiglu_fixup_kernel sums the parts, a = silu(h1)*h3
//   pass 2   partial gate * W2_e a             -> combine kernel sums parts and slots into y
//
// Same warp roles, barriers and bounded waits as the training-shaped kernel: warp 0 TMA producer
// (128x64 weights + 32, 64 or 128 x 64 tokens per CTA and stage; 9, 8 or 6 stages), warp 1 MMA issuer in the leader CTA,
// warps 2-9 epilogue.
#include "btx_tc_ptx.cuh"

namespace btx {
namespace {

using namespace tcx;

constexpr int WM = 128;                                  // weight rows per CTA (256 per pair)
constexpr int CH = kRowTile;                             // a chunk is one padded row tile of an expert (MMA N <= 256)
constexpr int D_MAX_STAGES = 9;
constexpr int DA_BYTES = WM * BK * 2;                    // weights per CTA and stage
constexpr int D_RING_BYTES = 192 * 1024;                 // stages = min(9, ring / (DA_BYTES + token box))
constexpr int D_EPI_WARPS = 8;
constexpr int D_THREADS = 64 + D_EPI_WARPS * 32;
constexpr int D_MAX_CHUNKS = 72;                         // row tiles that can hold tokens: at most R/256 + E = 4 + 64
constexpr int D_SMEM_BYTES = D_RING_BYTES + 1024 + 256 + (D_MAX_CHUNKS + 2) * 4;

struct SwapParams {
  int W;                        // weight rows per expert (F in pass 1, d in pass 2)
  int E, S, n_w, m_tiles, kb_total;
  int box_rows;                 // token rows each CTA loads per stage (32, 64 or 128): >= N/2 of every chunk
  int stages;                   // ring depth for that box
  const int32_t* pad_offsets;
  const int32_t* tile_expert;
  const int32_t* counts;        // rows per expert
  const int32_t* rowmap;
  const float* gates;           // non-null: scale every token column by its gate
  float* out0;                  // [S][R][W]
  float* out1;                  // second weight matrix (pass 1: W3)
  size_t split_stride;          // R * W
  int32_t* status;
};

struct DTile { int which, chunk, n, mt, e, kb0, kb1, s; };   // n = MMA N of the chunk (multiple of 16)

__device__ __forceinline__ DTile d_tile(const SwapParams& p, const int* chunks, int n_valid, int t) {
  // The token chunk varies fastest: an expert that holds more than one chunk of tokens has the items
  // that read the same weight tile next to one another, so the tile comes from HBM once and from L2
  // for the other chunks.
  DTile tl;
  const int ci = t % n_valid; t /= n_valid;
  tl.s = t % p.S; t /= p.S;
  tl.mt = t % p.m_tiles;
  tl.which = t / p.m_tiles;
  tl.chunk = chunks[ci] & 0xFFFF;
  tl.n = chunks[ci] >> 16;
  tl.e = p.tile_expert[tl.chunk];
  tl.kb0 = (int)((long long)tl.s * p.kb_total / p.S);
  tl.kb1 = (int)((long long)(tl.s + 1) * p.kb_total / p.S);
  return tl;
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(D_THREADS, 1)
tc_swapk_kernel(const __grid_constant__ CUtensorMap tmW0, const __grid_constant__ CUtensorMap tmW1,
                const __grid_constant__ CUtensorMap tmX, const SwapParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t ring = (raw + 1023u) & ~1023u;
  uint8_t* ctl = smem_raw + (ring - raw) + D_RING_BYTES;
  const uint32_t bar_full = smem_u32(ctl);
  const uint32_t bar_empty = bar_full + D_MAX_STAGES * 8;
  const uint32_t bar_tfull = bar_empty + D_MAX_STAGES * 8;
  const uint32_t bar_tempty = bar_tfull + 16;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ctl + D_MAX_STAGES * 16 + 32);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ctl + D_MAX_STAGES * 16 + 40);
  int* chunks = reinterpret_cast<int*>(ctl + 256);        // [0] = count, [1..] = chunk id | N << 16 of the chunks with tokens
  const int n_stages = p.stages;
  const uint32_t stage_bytes = DA_BYTES + (uint32_t)p.box_rows * (BK * 2);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  allow_dependents();

  if (threadIdx.x == 0) {
    for (int s = 0; s < D_MAX_STAGES; ++s) { mbar_init(bar_full + s * 8, 1); mbar_init(bar_empty + s * 8, 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(bar_tfull + a * 8, 1); mbar_init(bar_tempty + a * 8, 2 * D_EPI_WARPS * 32); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  // Barriers and TMEM are set up while the kernel before this one may still run; everything below
  // reads what it wrote.
  grid_dependency_wait();
  if (warp == 0) {
    // List of the chunks (row tiles) that hold tokens, each with its MMA N: an expert's segment starts
    // with its real rows, so tile j of expert e holds min(256, counts[e] - 256 j) of them.  The 32
    // lanes probe 32 tiles at a time: one round of global-memory latency, not one per tile.
    __syncwarp();
    const int all = p.pad_offsets[p.E] / CH;
    int n = 0;
    for (int c0 = 0; c0 < all; c0 += 32) {
      const int c = c0 + lane;
      int rows = 0;
      if (c < all) {
        const int e = p.tile_expert[c];
        if (e >= 0) rows = min(CH, p.counts[e] - (c * CH - p.pad_offsets[e]));
      }
      const bool holds = rows > 0;
      const unsigned m = __ballot_sync(0xffffffffu, holds);
      const int pos = n + __popc(m & ((1u << lane) - 1u));
      if (holds && pos < D_MAX_CHUNKS) chunks[1 + pos] = c | (((rows + 15) & ~15) << 16);
      n += __popc(m);
    }
    if (lane == 0) chunks[0] = min(n, D_MAX_CHUNKS);
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
  const int n_valid = chunks[0];
  const int n_total = p.n_w * n_valid * p.m_tiles * p.S;

  if (warp == 0) {
    if (lane == 0) {
      uint32_t stage = 0, phase = 0;
      bool ok = true;
      for (int t = pair; t < n_total && ok; t += n_pairs) {
        const DTile tl = d_tile(p, chunks + 1, n_valid, t);
        for (int kb = tl.kb0; kb < tl.kb1; ++kb) {
          if (!(ok = mbar_wait(bar_empty + stage * 8, phase ^ 1u, abort_flag, p.status))) break;
          const uint32_t full_local = bar_full + stage * 8;
          const uint32_t full = map_to_cta(full_local, 0);
          const uint32_t sA = ring + stage * stage_bytes, sB = sA + DA_BYTES;
          if (rank == 0) mbar_expect_tx(full_local, 2 * stage_bytes);
          tma_load_3d(sA, tl.which ? &tmW1 : &tmW0, kb * BK, tl.mt * 2 * WM + (int)rank * WM, tl.e, full);
          // this CTA's half of the chunk's N token rows leads its box; rows past it are not used
          tma_load_2d(sB, &tmX, kb * BK, tl.chunk * CH + (int)rank * (tl.n / 2), full);
          if (++stage == n_stages) { stage = 0; phase ^= 1u; }
        }
      }
      for (int i = 0; i < n_stages && ok; ++i) {          // drain: all commits to this CTA have landed
        ok = mbar_wait(bar_empty + stage * 8, phase ^ 1u, abort_flag, p.status);
        if (++stage == n_stages) { stage = 0; phase ^= 1u; }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc_base = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)((2 * WM) >> 4) << 24);
      uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
      bool ok = true;
      for (int t = pair; t < n_total && ok; t += n_pairs) {
        const DTile tl = d_tile(p, chunks + 1, n_valid, t);
        if (tl.kb1 <= tl.kb0) continue;
        if (!(ok = mbar_wait(bar_tempty + acc * 8, acc_phase ^ 1u, abort_flag, p.status))) break;
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + acc * 256;
        const uint32_t idesc = idesc_base | ((uint32_t)(tl.n >> 3) << 17);
        for (int kb = tl.kb0; kb < tl.kb1; ++kb) {
          if (!(ok = mbar_wait(bar_full + stage * 8, phase, abort_flag, p.status))) break;
          tc_fence_after();
          const uint32_t sA = ring + stage * stage_bytes, sB = sA + DA_BYTES;
          const uint64_t da = smem_desc(sA, false), db = smem_desc(sB, false);
#pragma unroll
          for (int k16 = 0; k16 < BK / 16; ++k16)
            tc_mma_pair(tmem_d, da + (uint64_t)(2 * k16), db + (uint64_t)(2 * k16), idesc,
                        (kb > tl.kb0 || k16 > 0) ? 1u : 0u);
          tc_commit_pair(bar_empty + stage * 8);
          if (++stage == n_stages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tc_commit_pair(bar_tfull + acc * 8);
        acc ^= 1u;
        if (acc == 0) acc_phase ^= 1u;
      }
    }
  } else {
    const int q = warp & 3, half = (warp - 2) >> 2;
    const uint32_t tempty_leader = map_to_cta(bar_tempty, 0);
    uint32_t acc = 0, acc_phase = 0;
    bool ok = true;
    for (int t = pair; t < n_total && ok; t += n_pairs) {
      const DTile tl = d_tile(p, chunks + 1, n_valid, t);
      if (tl.kb1 <= tl.kb0) continue;
      if (!(ok = mbar_wait(bar_tfull + acc * 8, acc_phase, abort_flag, p.status))) break;
      tc_fence_after();
      const int wrow = tl.mt * 2 * WM + (int)rank * WM + q * 32 + lane;
      float* out = (tl.which ? p.out1 : p.out0) + (size_t)tl.s * p.split_stride + wrow;
      // the two warps of a lane quarter take alternate groups of 32 token columns
      for (int c0 = half * 32; c0 < tl.n; c0 += 64) {
        // token of this lane's column: lane i of the warp looks up column c0 + i
        const int my_flat = p.rowmap[tl.chunk * CH + c0 + lane];
        const float my_gate = (p.gates != nullptr && my_flat >= 0) ? p.gates[my_flat] : 1.0f;
        float v[32];
        tc_ld32(tmem_base + acc * 256 + c0 + ((uint32_t)(q * 32) << 16), v);
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const int flat = __shfl_sync(0xffffffffu, my_flat, i);
          const float g = __shfl_sync(0xffffffffu, my_gate, i);
          if (flat >= 0 && wrow < p.W) out[(size_t)flat * p.W] = g * v[i];
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

// act[row][f] = silu(sum_s P1) * (sum_s P3) for the rows that hold tokens; h1/h3 are kept as well
// when the forward saves for backward.  One block row per assignment, four columns per thread.
__global__ void __launch_bounds__(256)
swiglu_fixup_kernel(int F, int S, size_t split_stride, const float* __restrict__ p1, const float* __restrict__ p3,
                    const int32_t* __restrict__ flat2row, __nv_bfloat16* __restrict__ act,
                    __nv_bfloat16* __restrict__ h1s, __nv_bfloat16* __restrict__ h3s) {
  const int flat = blockIdx.y;
  const int f = (blockIdx.x * blockDim.x + threadIdx.x) * 4;
  allow_dependents();
  grid_dependency_wait();
  if (f >= F || flat2row[flat] < 0) return;          // a dropped assignment holds no row
  const size_t src = (size_t)flat * F + f;
  float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
  for (int s = 0; s < S; ++s) {
    const float4 x = *reinterpret_cast<const float4*>(p1 + s * split_stride + src);
    const float4 y = *reinterpret_cast<const float4*>(p3 + s * split_stride + src);
    a.x += x.x; a.y += x.y; a.z += x.z; a.w += x.w;
    b.x += y.x; b.y += y.y; b.z += y.z; b.w += y.w;
  }
  auto pack4 = [](float x0, float x1, float x2, float x3) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(x0, x1), hi = __floats2bfloat162_rn(x2, x3);
    return make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
  };
  const size_t dst = (size_t)flat2row[flat] * F + f;
  *reinterpret_cast<uint2*>(act + dst) =
      pack4(fast_swiglu(a.x, b.x), fast_swiglu(a.y, b.y), fast_swiglu(a.z, b.z), fast_swiglu(a.w, b.w));
  if (h1s != nullptr) {
    *reinterpret_cast<uint2*>(h1s + dst) = pack4(a.x, a.y, a.z, a.w);
    *reinterpret_cast<uint2*>(h3s + dst) = pack4(b.x, b.y, b.z, b.w);
  }
}

btx_status launch_swapk(const CUtensorMap& w0, const CUtensorMap& w1, const CUtensorMap& x, const SwapParams& p,
                        cudaStream_t st) {
  if (cudaFuncSetAttribute(tc_swapk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, D_SMEM_BYTES) != cudaSuccess)
    return BTX_ERR_CUDA;
  int pairs = sm_count() / 2;
  if (pairs < 1) pairs = 1;
  return launch_after_predecessor(tc_swapk_kernel, dim3(2 * pairs), dim3(D_THREADS), D_SMEM_BYTES, st, true, w0, w1, x,
                                  p) == cudaSuccess ? BTX_OK : BTX_ERR_CUDA;
}

}  // namespace

// Smallest number of contraction splits with which base_tiles * S work items keep at least 85 % of
// the CTA pairs busy in every round.  That is enough to saturate HBM: at the Llama-2-7B shape one
// un-split round of 64 items on 74 pairs streams W2 as fast as 512 items in seven rounds did, and
// fewer splits mean fewer partial products to write and to sum.
int pick_decode_splits(int base_tiles, int kb_total) {
  const int pairs = sm_count() / 2 > 0 ? sm_count() / 2 : 1;
  int best = 1;
  double best_eff = 0.0;
  for (int S = 1; S <= 8 && S <= kb_total; ++S) {
    const int tiles = base_tiles * S;
    const double eff = (double)tiles / (double)(((tiles + pairs - 1) / pairs) * pairs);
    if (eff > best_eff + 1e-9) { best_eff = eff; best = S; }
    if (eff >= 0.85) return S;
  }
  return best;
}

btx_status launch_expert_forward_small_bf16(const Plan& pl, const void* w1, const void* w3, const void* w2,
                                            const Buffers& b, int save, cudaStream_t st) {
  const uint64_t d = pl.d, F = pl.F, E = pl.E, RP = pl.r_pad_max;
  CUtensorMap m0, m1, mx;
  btx_status s;
  SwapParams p = {};
  p.E = pl.E; p.pad_offsets = b.pad_offsets; p.tile_expert = b.tile_expert; p.rowmap = b.rowmap; p.status = b.status;
  p.counts = b.counts;
  // a chunk holds at most min(T, 256) tokens (a token meets an expert once): each CTA loads half of them
  const int n_max = ((pl.T < CH ? pl.T : CH) + 15) & ~15;
  p.box_rows = n_max / 2 <= 32 ? 32 : (n_max / 2 <= 64 ? 64 : 128);
  p.stages = D_RING_BYTES / (DA_BYTES + p.box_rows * BK * 2);
  if (p.stages > D_MAX_STAGES) p.stages = D_MAX_STAGES;
  if (save) {   // backward reads whole padded tiles of h1/h3: rows without a token must be finite
    if (cudaMemsetAsync(b.h1, 0, (size_t)RP * F * 2, st) != cudaSuccess ||
        cudaMemsetAsync(b.h3, 0, (size_t)RP * F * 2, st) != cudaSuccess)
      return BTX_ERR_CUDA;
  }
  // pass 1: partial h1, h3
  if (!make_map(&m0, w1, d, F, E, 64, WM) || !make_map(&m1, w3, d, F, E, 64, WM) || !make_map(&mx, b.xs, d, RP, 0, 64, p.box_rows))
    return BTX_ERR_CUDA;
  p.W = pl.F; p.n_w = 2; p.m_tiles = (pl.F + 2 * WM - 1) / (2 * WM); p.kb_total = (pl.d + BK - 1) / BK; p.S = pl.dec_s1;
  p.split_stride = (size_t)pl.R * pl.F;
  p.out0 = b.part; p.out1 = b.part + (size_t)pl.dec_s1 * p.split_stride; p.gates = nullptr;
  if ((s = launch_swapk(m0, m1, mx, p, st)) != BTX_OK) return s;
  if (launch_after_predecessor(swiglu_fixup_kernel, dim3((pl.F / 4 + 255) / 256, pl.R), dim3(256), 0, st, true, pl.F,
                               pl.dec_s1, p.split_stride, (const float*)p.out0, (const float*)p.out1,
                               (const int32_t*)b.flat2row, (__nv_bfloat16*)b.act,
                               save ? (__nv_bfloat16*)b.h1 : (__nv_bfloat16*)nullptr,
                               save ? (__nv_bfloat16*)b.h3 : (__nv_bfloat16*)nullptr) != cudaSuccess)
    return BTX_ERR_CUDA;
  mark_stage(2, st);
  // pass 2: partial gate-scaled expert rows
  if (!make_map(&m0, w2, F, d, E, 64, WM) || !make_map(&mx, b.act, F, RP, 0, 64, p.box_rows)) return BTX_ERR_CUDA;
  p.W = pl.d; p.n_w = 1; p.m_tiles = (pl.d + 2 * WM - 1) / (2 * WM); p.kb_total = (pl.F + BK - 1) / BK; p.S = pl.dec_s2;
  p.split_stride = (size_t)pl.R * pl.d;
  p.out0 = b.part; p.out1 = b.part; p.gates = b.gates;
  return launch_swapk(m0, m0, mx, p, st);
}

}  // namespace btx
