// FP32 expert GEMMs on the plain ALUs (FFMA), used by BTX_F32 mode where a 1e-5 tolerance
// rules out reduced-precision tensor-core inputs.  Same data flow and fused epilogues as the
// tensor-core path: SwiGLU in the W1/W3 epilogue, gate-scaled row scatter in the W2 epilogue,
// SwiGLU backward + gate row-dot in the dgrad-2 epilogue, contraction over tokens for wgrad.
#include "btx_common.cuh"

namespace btx {
namespace {

constexpr int TM = 64, TN = 64, TK = 16;

enum SimtMode { S_FWD1 = 0, S_FWD2 = 1, S_DACT = 2, S_DX = 3, S_WGRAD = 4 };

struct SimtParams {
  int d, F, E, r_pad_max;
  const int32_t* tile_expert;   // per 128-row tile of the padded layout
  const int32_t* pad_offsets;
  const int32_t* rowmap;
  const float* gates;           // [R] by flat assignment id
  const float* a0;              // A operand(s)
  const float* a1;
  const float* b0;              // B operand(s)
  const float* b1;
  const float* h1;              // saved pre-activations (DACT)
  const float* h3;
  float* o0;                    // outputs
  float* o1;
  float* o2;
  float* dg_part;
  int save, accumulate;
  int M, N;                     // WGRAD: output rows / cols per expert; others: N = output cols
  int ldp, ldq;                 // WGRAD operand row strides
};

template <int MODE>
__global__ void __launch_bounds__(256) simt_gemm_kernel(SimtParams p) {
  __shared__ float As[TK][TM + 1];
  __shared__ float Bs[TK][TN + 1];
  __shared__ float Bs2[(MODE == S_FWD1) ? TK : 1][TN + 1];
  __shared__ float rowred[(MODE == S_DACT) ? TM : 1][17];

  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int n0 = blockIdx.x * TN;
  const int m0 = blockIdx.y * TM;
  int e, k_begin = 0, K;
  if (MODE == S_WGRAD) {
    e = blockIdx.z;
    k_begin = p.pad_offsets[e];
    K = p.pad_offsets[e + 1] - k_begin;
  } else {
    if (m0 >= p.pad_offsets[p.E]) return;
    e = p.tile_expert[m0 / kRowTile];
    K = (MODE == S_FWD1 || MODE == S_DACT) ? p.d : (MODE == S_FWD2 ? p.F : 2 * p.F);
  }
  const int d = p.d, F = p.F;
  const int Mlim = (MODE == S_WGRAD) ? p.M : p.pad_offsets[p.E];
  const int Nlim = p.N;

  auto loadA = [&](int m, int kk) -> float {
    if (m >= Mlim || kk >= K) return 0.f;
    if (MODE == S_FWD1 || MODE == S_DACT) return p.a0[(size_t)m * d + kk];
    if (MODE == S_FWD2) return p.a0[(size_t)m * F + kk];
    if (MODE == S_DX) return kk < F ? p.a0[(size_t)m * F + kk] : p.a1[(size_t)m * F + kk - F];
    return p.a0[(size_t)(k_begin + kk) * p.ldp + m];
  };
  auto loadB = [&](int n, int kk, int which) -> float {
    if (n >= Nlim || kk >= K) return 0.f;
    if (MODE == S_FWD1) return (which ? p.b1 : p.b0)[((size_t)e * F + n) * d + kk];
    if (MODE == S_FWD2) return p.b0[((size_t)e * d + n) * F + kk];
    if (MODE == S_DACT) return p.b0[((size_t)e * d + kk) * F + n];
    if (MODE == S_DX) return kk < F ? p.b0[((size_t)e * F + kk) * d + n] : p.b1[((size_t)e * F + kk - F) * d + n];
    return p.b0[(size_t)(k_begin + kk) * p.ldq + n];
  };

  float acc[4][4], acc2[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = acc2[i][j] = 0.f;

  for (int k0 = 0; k0 < K; k0 += TK) {
    // operands whose contraction index is contiguous are read with kk fastest, others with m/n fastest
    constexpr bool a_k_contig = (MODE != S_WGRAD);
    constexpr bool b_k_contig = (MODE == S_FWD1 || MODE == S_FWD2);
    for (int i = threadIdx.x; i < TM * TK; i += 256) {
      int kk = a_k_contig ? (i % TK) : (i / TM), m = a_k_contig ? (i / TK) : (i % TM);
      As[kk][m] = loadA(m0 + m, k0 + kk);
    }
    for (int i = threadIdx.x; i < TN * TK; i += 256) {
      int kk = b_k_contig ? (i % TK) : (i / TN), n = b_k_contig ? (i / TK) : (i % TN);
      Bs[kk][n] = loadB(n0 + n, k0 + kk, 0);
      if (MODE == S_FWD1) Bs2[kk][n] = loadB(n0 + n, k0 + kk, 1);
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < TK; ++kk) {
      float a[4], b[4], b2[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        b[j] = Bs[kk][tx * 4 + j];
        b2[j] = (MODE == S_FWD1) ? Bs2[kk][tx * 4 + j] : 0.f;
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
          if (MODE == S_FWD1) acc2[i][j] = fmaf(a[i], b2[j], acc2[i][j]);
        }
    }
    __syncthreads();
  }

  // ---- epilogues ----
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    float rowdot = 0.f;
    if (m < Mlim) {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int n = n0 + tx * 4 + j;
        if (n >= Nlim) continue;
        const float v = acc[i][j];
        if (MODE == S_FWD1) {
          const float h1 = v, h3 = acc2[i][j];
          p.o0[(size_t)m * F + n] = swiglu_f32(h1, h3);
          if (p.save) { p.o1[(size_t)m * F + n] = h1; p.o2[(size_t)m * F + n] = h3; }
        } else if (MODE == S_FWD2) {
          const int flat = p.rowmap[m];
          if (flat >= 0) p.o0[(size_t)flat * d + n] = p.gates[flat] * v;
        } else if (MODE == S_DACT) {
          const int flat = p.rowmap[m];
          const float g = flat >= 0 ? p.gates[flat] : 0.f;
          const float h1 = p.h1[(size_t)m * F + n], h3 = p.h3[(size_t)m * F + n];
          const float a = swiglu_f32(h1, h3);
          float dh1, dh3;
          swiglu_bwd_f32(h1, h3, g * v, dh1, dh3);
          p.o0[(size_t)m * F + n] = dh1;
          p.o1[(size_t)m * F + n] = dh3;
          p.o2[(size_t)m * F + n] = g * a;
          rowdot += v * a;
        } else if (MODE == S_DX) {
          const int flat = p.rowmap[m];
          if (flat >= 0) p.o0[(size_t)flat * d + n] = v;
        } else {
          float* o = p.o0 + ((size_t)e * p.M + m) * p.N + n;
          *o = p.accumulate ? *o + v : v;
        }
      }
    }
    if (MODE == S_DACT) rowred[ty * 4 + i][tx] = rowdot;
  }
  if (MODE == S_DACT) {
    __syncthreads();
    if (threadIdx.x < TM) {
      float s = 0.f;
      for (int j = 0; j < 16; ++j) s += rowred[threadIdx.x][j];
      int m = m0 + threadIdx.x;
      if (m < Mlim) p.dg_part[(size_t)blockIdx.x * p.r_pad_max + m] = s;
    }
  }
}

}  // namespace

cudaError_t launch_expert_forward_f32(const Plan& pl, const void* w1, const void* w3, const void* w2,
                                      const Buffers& b, int save, cudaStream_t st) {
  SimtParams p = {};
  p.d = pl.d; p.F = pl.F; p.E = pl.E; p.r_pad_max = pl.r_pad_max;
  p.tile_expert = b.tile_expert; p.pad_offsets = b.pad_offsets; p.rowmap = b.rowmap; p.gates = b.gates;
  const int mt = pl.r_pad_max / TM;
  // GEMM-1: h1 = Xs W1^T, h3 = Xs W3^T, act = silu(h1) * h3
  p.a0 = (const float*)b.xs; p.b0 = (const float*)w1; p.b1 = (const float*)w3;
  p.o0 = (float*)b.act; p.o1 = (float*)b.h1; p.o2 = (float*)b.h3; p.save = save; p.N = pl.F;
  simt_gemm_kernel<S_FWD1><<<dim3((pl.F + TN - 1) / TN, mt), 256, 0, st>>>(p);
  mark_stage(2, st);
  // GEMM-2: gate-scaled expert rows
  p.a0 = (const float*)b.act; p.b0 = (const float*)w2; p.o0 = b.yp; p.N = pl.d;
  simt_gemm_kernel<S_FWD2><<<dim3((pl.d + TN - 1) / TN, mt), 256, 0, st>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_expert_backward_f32(const Plan& pl, const void* w1, const void* w3, const void* w2,
                                       const Buffers& b, float* dw1, float* dw3, float* dw2, int accumulate,
                                       int skip_wgrad, cudaEvent_t after_dx, cudaStream_t st) {
  SimtParams p = {};
  p.d = pl.d; p.F = pl.F; p.E = pl.E; p.r_pad_max = pl.r_pad_max;
  p.tile_expert = b.tile_expert; p.pad_offsets = b.pad_offsets; p.rowmap = b.rowmap; p.gates = b.gates;
  p.accumulate = accumulate;
  const int mt = pl.r_pad_max / TM;
  // dgrad-2 + SwiGLU backward: dA' = dYs W2
  p.a0 = (const float*)b.dys; p.b0 = (const float*)w2; p.h1 = (const float*)b.h1; p.h3 = (const float*)b.h3;
  p.o0 = (float*)b.dh1; p.o1 = (float*)b.dh3; p.o2 = (float*)b.ga; p.dg_part = b.dg_part; p.N = pl.F;
  simt_gemm_kernel<S_DACT><<<dim3((pl.F + TN - 1) / TN, mt), 256, 0, st>>>(p);
  mark_stage(2, st);
  // dgrad-1: dXs = dh1 W1 + dh3 W3
  p.a0 = (const float*)b.dh1; p.a1 = (const float*)b.dh3; p.b0 = (const float*)w1; p.b1 = (const float*)w3;
  p.o0 = b.dxp; p.N = pl.d;
  simt_gemm_kernel<S_DX><<<dim3((pl.d + TN - 1) / TN, mt), 256, 0, st>>>(p);
  mark_stage(3, st);
  if (after_dx != nullptr) cudaEventRecord(after_dx, st);      // the router backward may start here
  if (skip_wgrad) return cudaGetLastError();
  // wgrads: contraction over the expert's (padded) token rows
  p.a0 = (const float*)b.dys; p.ldp = pl.d; p.b0 = (const float*)b.ga; p.ldq = pl.F; p.o0 = dw2; p.M = pl.d; p.N = pl.F;
  simt_gemm_kernel<S_WGRAD><<<dim3((pl.F + TN - 1) / TN, (pl.d + TM - 1) / TM, pl.E), 256, 0, st>>>(p);
  mark_stage(4, st);
  p.a0 = (const float*)b.dh1; p.ldp = pl.F; p.b0 = (const float*)b.xs; p.ldq = pl.d; p.o0 = dw1; p.M = pl.F; p.N = pl.d;
  simt_gemm_kernel<S_WGRAD><<<dim3((pl.d + TN - 1) / TN, (pl.F + TM - 1) / TM, pl.E), 256, 0, st>>>(p);
  mark_stage(5, st);
  p.a0 = (const float*)b.dh3; p.o0 = dw3;
  simt_gemm_kernel<S_WGRAD><<<dim3((pl.d + TN - 1) / TN, (pl.F + TM - 1) / TM, pl.E), 256, 0, st>>>(p);
  mark_stage(6, st);
  return cudaGetLastError();
}

}  // namespace btx
