// MiX merge (Section 3.2): feed-forward matrices are copied into the stacked expert tensor,
// every other parameter is averaged over the N models.  One persistent, bandwidth-bound kernel
// walks a table of work items in 64 KB chunks with 128-bit streaming loads and stores, four
// vectors per thread in flight from every source.
#include <vector>

#include "btx_common.cuh"

namespace btx {
namespace {

constexpr int kMaxModels = 16;
constexpr int kChunkVecs = 4096;          // 16-byte vectors per chunk (64 KB of output)
constexpr int kMergeThreads = 256;

struct DevItem {
  uint64_t numel;
  void* dst;
  int32_t nsrc;                           // 1: copy, N: average
  uint32_t row_vecs;                      // copies only: 0 = linear, else 16-byte vectors per row of a 2-D block
  uint32_t src_pitch, dst_pitch;          // row pitches of the block in 16-byte vectors
  const void* src[kMaxModels];
};

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ void st_stream(uint4* p, uint4 v) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

template <typename T> struct Elem;
template <> struct Elem<float> {
  static constexpr int PER_VEC = 4;
  static __device__ __forceinline__ void add(float (&acc)[8], uint4 v) {
    acc[0] += __uint_as_float(v.x); acc[1] += __uint_as_float(v.y);
    acc[2] += __uint_as_float(v.z); acc[3] += __uint_as_float(v.w);
  }
  static __device__ __forceinline__ uint4 pack(const float (&acc)[8], float n) {
    return make_uint4(__float_as_uint(acc[0] / n), __float_as_uint(acc[1] / n), __float_as_uint(acc[2] / n),
                      __float_as_uint(acc[3] / n));
  }
};
template <> struct Elem<__nv_bfloat16> {
  static constexpr int PER_VEC = 8;
  static __device__ __forceinline__ void add(float (&acc)[8], uint4 v) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      acc[2 * i] += __uint_as_float(w[i] << 16);           // low half = even element
      acc[2 * i + 1] += __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  static __device__ __forceinline__ uint4 pack(const float (&acc)[8], float n) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      __nv_bfloat162 h = __floats2bfloat162_rn(acc[2 * i] / n, acc[2 * i + 1] / n);
      w[i] = *reinterpret_cast<uint32_t*>(&h);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
  }
};

template <typename T>
__global__ void __launch_bounds__(kMergeThreads)
merge_kernel(const DevItem* __restrict__ items, const uint64_t* __restrict__ chunk_start, int n_items,
             uint64_t total_chunks) {
  __shared__ DevItem it;
  __shared__ uint64_t first_chunk;
  for (uint64_t c = blockIdx.x; c < total_chunks; c += gridDim.x) {
    __syncthreads();
    if (threadIdx.x == 0) {
      int lo = 0, hi = n_items - 1;                         // last item whose first chunk <= c
      while (lo < hi) {
        int mid = (lo + hi + 1) >> 1;
        if (chunk_start[mid] <= c) lo = mid; else hi = mid - 1;
      }
      it = items[lo];
      first_chunk = chunk_start[lo];
    }
    __syncthreads();
    const uint64_t nvec = it.numel / Elem<T>::PER_VEC;
    const uint64_t v0 = (c - first_chunk) * kChunkVecs;
    const uint64_t v1 = min(nvec, v0 + (uint64_t)kChunkVecs);
    const int ns = it.nsrc;
    uint4* dst = reinterpret_cast<uint4*>(it.dst);
    constexpr int U = 4;                                    // vectors per thread per round
    if (ns == 1 && it.row_vecs != 0) {
      // 2-D block copy (a column range of W2, or a row range placed inside a wider tensor)
      const uint4* s = reinterpret_cast<const uint4*>(it.src[0]);
      const uint32_t rv = it.row_vecs;
      for (uint64_t v = v0 + threadIdx.x; v < v1; v += kMergeThreads) {
        const uint64_t r = v / rv, cidx = v - r * rv;
        st_stream(dst + r * it.dst_pitch + cidx, ld_stream(s + r * it.src_pitch + cidx));
      }
    } else if (ns == 1) {
      const uint4* s = reinterpret_cast<const uint4*>(it.src[0]);
      uint64_t v = v0 + threadIdx.x;
      for (; v + (U - 1) * kMergeThreads < v1; v += U * kMergeThreads) {
        uint4 x[U];
#pragma unroll
        for (int u = 0; u < U; ++u) x[u] = ld_stream(s + v + u * kMergeThreads);
#pragma unroll
        for (int u = 0; u < U; ++u) st_stream(dst + v + u * kMergeThreads, x[u]);
      }
      for (; v < v1; v += kMergeThreads) st_stream(dst + v, ld_stream(s + v));
    } else if (ns == 4) {
      // the common case (four expert LLMs): all 16 loads of a round are issued before any use
      const uint4* s0 = reinterpret_cast<const uint4*>(it.src[0]);
      const uint4* s1 = reinterpret_cast<const uint4*>(it.src[1]);
      const uint4* s2 = reinterpret_cast<const uint4*>(it.src[2]);
      const uint4* s3 = reinterpret_cast<const uint4*>(it.src[3]);
      uint64_t v = v0 + threadIdx.x;
      for (; v + (U - 1) * kMergeThreads < v1; v += U * kMergeThreads) {
        uint4 x[U][4];
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const uint64_t w = v + u * kMergeThreads;
          x[u][0] = ld_stream(s0 + w); x[u][1] = ld_stream(s1 + w); x[u][2] = ld_stream(s2 + w); x[u][3] = ld_stream(s3 + w);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
          float acc[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) acc[i] = 0.f;
#pragma unroll
          for (int m = 0; m < 4; ++m) Elem<T>::add(acc, x[u][m]);    // model order 0..3
          st_stream(dst + v + u * kMergeThreads, Elem<T>::pack(acc, 4.0f));
        }
      }
      for (; v < v1; v += kMergeThreads) {
        float acc[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] = 0.f;
        Elem<T>::add(acc, ld_stream(s0 + v)); Elem<T>::add(acc, ld_stream(s1 + v));
        Elem<T>::add(acc, ld_stream(s2 + v)); Elem<T>::add(acc, ld_stream(s3 + v));
        st_stream(dst + v, Elem<T>::pack(acc, 4.0f));
      }
    } else {
      for (uint64_t v = v0 + threadIdx.x; v < v1; v += kMergeThreads) {
        float acc[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] = 0.f;
        for (int m = 0; m < ns; ++m) Elem<T>::add(acc, ld_stream(reinterpret_cast<const uint4*>(it.src[m]) + v));
        st_stream(dst + v, Elem<T>::pack(acc, (float)ns));
      }
    }
    // elements past the last whole vector: done by the block that owns the item's last chunk
    if (v1 == nvec) {
      const uint64_t tail0 = nvec * Elem<T>::PER_VEC;
      for (uint64_t i = tail0 + threadIdx.x; i < it.numel; i += kMergeThreads) {
        T* d = reinterpret_cast<T*>(it.dst);
        if (ns == 1) {
          d[i] = reinterpret_cast<const T*>(it.src[0])[i];
        } else {
          float a = 0.f;
          for (int m = 0; m < ns; ++m) a += to_f32(reinterpret_cast<const T*>(it.src[m])[i]);
          d[i] = from_f32<T>(a / (float)ns);
        }
      }
    }
  }
}

uint64_t chunks_of(uint64_t numel, int per_vec) {
  uint64_t nvec = numel / per_vec;
  uint64_t c = (nvec + kChunkVecs - 1) / kChunkVecs;
  return c == 0 ? 1 : c;
}

}  // namespace
}  // namespace btx

using namespace btx;

static btx_status launch_merge_items(std::vector<DevItem>& dev, std::vector<uint64_t>& start, uint64_t total,
                                     int32_t dtype, void* workspace, size_t workspace_bytes, void* stream) {
  if (dev.empty()) return BTX_OK;
  start.push_back(total);
  const size_t need = kStatusWords * 4 + dev.size() * sizeof(DevItem) + start.size() * sizeof(uint64_t);
  if (workspace_bytes < need) return BTX_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  char* w = (char*)workspace + kStatusWords * 4;
  DevItem* d_items = (DevItem*)w;
  uint64_t* d_start = (uint64_t*)(w + dev.size() * sizeof(DevItem));
  // The tables are pageable host memory: cudaMemcpyAsync stages them before it returns (the vectors may
  // then go out of scope), which also means that these two copies block the host for a moment and that a
  // merge call must not be recorded into a CUDA graph (a replay would read the freed vectors).
  if (cudaMemcpyAsync(d_items, dev.data(), dev.size() * sizeof(DevItem), cudaMemcpyHostToDevice, st) != cudaSuccess)
    return BTX_ERR_CUDA;
  if (cudaMemcpyAsync(d_start, start.data(), start.size() * sizeof(uint64_t), cudaMemcpyHostToDevice, st) !=
      cudaSuccess)
    return BTX_ERR_CUDA;
  uint64_t grid = (uint64_t)sm_count() * 8;
  if (grid > total) grid = total;
  if (dtype == BTX_BF16)
    merge_kernel<__nv_bfloat16><<<(unsigned)grid, kMergeThreads, 0, st>>>(d_items, d_start, (int)dev.size(), total);
  else
    merge_kernel<float><<<(unsigned)grid, kMergeThreads, 0, st>>>(d_items, d_start, (int)dev.size(), total);
  return cudaGetLastError() == cudaSuccess ? BTX_OK : BTX_ERR_CUDA;
}

extern "C" btx_status btx_merge_workspace_size(int32_t n_models, uint64_t n_items, size_t* workspace_bytes) {
  if (!workspace_bytes || n_models < 1 || n_models > kMaxModels) return BTX_ERR_INVALID_ARG;
  uint64_t sub = n_items * (uint64_t)n_models;             // an FFN item becomes n_models copies
  *workspace_bytes = kStatusWords * 4 + sub * sizeof(DevItem) + (sub + 1) * sizeof(uint64_t) + 256;
  return BTX_OK;
}

extern "C" btx_status btx_merge(int32_t n_models, int32_t dtype, const btx_merge_item* items, uint64_t n_items,
                                void* workspace, size_t workspace_bytes, void* stream) {
  if (n_models < 1 || n_models > kMaxModels) return BTX_ERR_UNSUPPORTED;
  if (dtype != BTX_F32 && dtype != BTX_BF16) return BTX_ERR_INVALID_ARG;
  if (n_items == 0) return BTX_OK;
  if (!items || !workspace) return BTX_ERR_INVALID_ARG;
  size_t need = 0;
  btx_merge_workspace_size(n_models, n_items, &need);
  if (workspace_bytes < need) return BTX_ERR_WORKSPACE;
  if (((uintptr_t)workspace & 15) != 0) return BTX_ERR_INVALID_ARG;
  const int esize = dtype == BTX_BF16 ? 2 : 4;
  const int per_vec = 16 / esize;

  std::vector<DevItem> dev;
  std::vector<uint64_t> start;
  uint64_t total = 0;
  for (uint64_t i = 0; i < n_items; ++i) {
    const btx_merge_item& it = items[i];
    if (!it.src || !it.dst || ((uintptr_t)it.dst & 15)) return BTX_ERR_INVALID_ARG;
    if (it.kind < BTX_PARAM_AVERAGE || it.kind > BTX_PARAM_FFN_W2) return BTX_ERR_INVALID_ARG;
    for (int m = 0; m < n_models; ++m)
      if (!it.src[m] || ((uintptr_t)it.src[m] & 15)) return BTX_ERR_INVALID_ARG;
    if (it.numel == 0) continue;
    if (it.kind == BTX_PARAM_AVERAGE) {
      DevItem d = {};
      d.numel = it.numel; d.dst = it.dst; d.nsrc = n_models;
      for (int m = 0; m < n_models; ++m) d.src[m] = it.src[m];
      dev.push_back(d); start.push_back(total); total += chunks_of(it.numel, per_vec);
    } else {
      if (n_models > 1 && (it.numel * esize) % 16 != 0) return BTX_ERR_UNSUPPORTED;   // stacked slots stay aligned
      for (int m = 0; m < n_models; ++m) {
        DevItem d = {};
        d.numel = it.numel; d.dst = (char*)it.dst + (size_t)m * it.numel * esize; d.nsrc = 1; d.src[0] = it.src[m];
        dev.push_back(d); start.push_back(total); total += chunks_of(it.numel, per_vec);
      }
    }
  }
  return launch_merge_items(dev, start, total, dtype, workspace, workspace_bytes, stream);
}

extern "C" btx_status btx_merge_ffn_workspace_size(int32_t n_models, int32_t chunks, size_t* workspace_bytes) {
  if (!workspace_bytes || n_models < 1 || n_models > kMaxModels || chunks < 1 || chunks > 64) return BTX_ERR_INVALID_ARG;
  const uint64_t c = chunks > n_models ? chunks : n_models;
  const uint64_t items = 3ull * n_models * c + 8;
  *workspace_bytes = kStatusWords * 4 + items * sizeof(DevItem) + (items + 1) * sizeof(uint64_t) + 256;
  return BTX_OK;
}

extern "C" btx_status btx_merge_ffn(int32_t n_models, int32_t dtype, int32_t layout, int32_t chunks, int32_t d_model,
                                    int32_t d_ff, const void* const* w1_src, const void* const* w3_src,
                                    const void* const* w2_src, void* w1_dst, void* w3_dst, void* w2_dst,
                                    void* workspace, size_t workspace_bytes, void* stream) {
  if (n_models < 1 || n_models > kMaxModels) return BTX_ERR_UNSUPPORTED;
  if (dtype != BTX_F32 && dtype != BTX_BF16) return BTX_ERR_INVALID_ARG;
  if (layout < BTX_FFN_STACK || layout > BTX_FFN_BLEND || d_model < 1 || d_ff < 1) return BTX_ERR_INVALID_ARG;
  if (!w1_src || !w3_src || !w2_src || !w1_dst || !w3_dst || !w2_dst || !workspace) return BTX_ERR_INVALID_ARG;
  const int C = layout == BTX_FFN_STACK ? 1 : (layout == BTX_FFN_BLEND ? n_models : chunks);
  if (C < 1 || d_ff % C != 0) return BTX_ERR_INVALID_ARG;
  const int esize = dtype == BTX_BF16 ? 2 : 4;
  const int per_vec = 16 / esize;
  const uint64_t Fc = (uint64_t)d_ff / C;                     // chunk width
  if ((Fc * esize) % 16 != 0 || ((uint64_t)d_model * esize) % 16 != 0) return BTX_ERR_UNSUPPORTED;
  auto bad = [](const void* p) { return p == nullptr || ((uintptr_t)p & 15) != 0; };
  if (bad(w1_dst) || bad(w3_dst) || bad(w2_dst) || ((uintptr_t)workspace & 15)) return BTX_ERR_INVALID_ARG;
  for (int m = 0; m < n_models; ++m)
    if (bad(w1_src[m]) || bad(w3_src[m]) || bad(w2_src[m])) return BTX_ERR_INVALID_ARG;

  std::vector<DevItem> dev;
  std::vector<uint64_t> start;
  uint64_t total = 0;
  auto push = [&](const void* src, void* dst, uint64_t numel, uint32_t row_elems, uint64_t src_pitch, uint64_t dst_pitch) {
    DevItem it = {};
    it.numel = numel; it.dst = dst; it.nsrc = 1; it.src[0] = src;
    if (row_elems != 0) {
      it.row_vecs = row_elems / per_vec; it.src_pitch = (uint32_t)(src_pitch / per_vec); it.dst_pitch = (uint32_t)(dst_pitch / per_vec);
    }
    dev.push_back(it); start.push_back(total); total += chunks_of(numel, per_vec);
  };
  const uint64_t d = d_model, F = d_ff;
  for (int i = 0; i < n_models; ++i) {
    const char* s1 = (const char*)w1_src[i]; const char* s3 = (const char*)w3_src[i]; const char* s2 = (const char*)w2_src[i];
    for (int c = 0; c < C; ++c) {
      // destination expert and, for BLEND, the slot of model i inside it
      const uint64_t e = layout == BTX_FFN_BLEND ? (uint64_t)c : (uint64_t)i * C + c;
      const uint64_t Fd = layout == BTX_FFN_BLEND ? F : Fc;                  // width of a destination expert
      const uint64_t slot = layout == BTX_FFN_BLEND ? (uint64_t)i * Fc : 0;   // first hidden unit inside the expert
      // W1/W3 [F, d]: rows c*Fc .. (c+1)*Fc of model i, contiguous
      const uint64_t src_rows = (uint64_t)c * Fc * d * esize;
      const uint64_t dst_rows = (e * Fd + slot) * d * esize;
      push(s1 + src_rows, (char*)w1_dst + dst_rows, Fc * d, 0, 0, 0);
      push(s3 + src_rows, (char*)w3_dst + dst_rows, Fc * d, 0, 0, 0);
      // W2 [d, F]: columns c*Fc .. (c+1)*Fc of model i -> columns slot .. slot+Fc of expert e
      push(s2 + (uint64_t)c * Fc * esize, (char*)w2_dst + (e * d * Fd + slot) * esize, d * Fc, (uint32_t)Fc, F, Fd);
    }
  }
  return launch_merge_items(dev, start, total, dtype, workspace, workspace_bytes, stream);
}
