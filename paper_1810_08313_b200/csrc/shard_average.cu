// Model averaging when the m replicas of a job are spread over G GPUs, m / G consecutive replicas on each
// (Section 2: the workers' models are averaged "by a fusion node or by performing an all-node broadcast";
// the paper's own runs used one worker per GPU).  One exchange per communication period:
//
//   1. partial_sum_kernel   on every GPU: p_g = x^(0) + x^(1) + ... over its own replicas, index order, fp32
//   2. the caller gathers the G partial sums into this GPU's own memory (an all-gather: NCCL, through the
//      callback of ls_set_shard; this library links no communication library and never reads a peer's memory)
//   3. combine_kernel       on every GPU: total = p_0 + p_1 + ... + p_{G-1} in rank order, mean = total / m,
//                           written to all local replicas (and their bf16 copies)
//
// The order (sequential inside a GPU, then sequential over the ranks) is fixed, so every GPU computes the same
// bits and all m replicas leave the step bitwise equal.  G = 1 is the arithmetic of average_kernel.
// Both kernels stream: one 32-byte slice per thread, every load of a slice issued before the first add.
#include "ls_internal.h"

namespace ls {
namespace {

constexpr int kThreads = 256;

struct V8 {
  float v[8];
  __device__ __forceinline__ void load(const float* p) {
    asm volatile("ld.global.L1::no_allocate.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7])
                 : "l"(p));
  }
  __device__ __forceinline__ void store(float* p) const {
    asm volatile("st.global.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "f"(v[0]), "f"(v[1]), "f"(v[2]),
                 "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7])
                 : "memory");
  }
};

// s = src[0] + src[1] + ... + src[n - 1] in that order (vectors `stride` floats apart), eight at a time in flight
__device__ __forceinline__ V8 ordered_sum(const float* src, int n, int64_t stride) {
  V8 s;
  s.load(src);
  for (int j0 = 1; j0 < n; j0 += 8) {
    V8 v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j)
      if (j0 + j < n) v[j].load(src + (int64_t)(j0 + j) * stride);
#pragma unroll
    for (int j = 0; j < 8; ++j)
      if (j0 + j < n)
#pragma unroll
        for (int e = 0; e < 8; ++e) s.v[e] = __fadd_rn(s.v[e], v[j].v[e]);
  }
  return s;
}
__device__ __forceinline__ float ordered_sum_scalar(const float* src, int n, int64_t stride) {
  float s = src[0];
  for (int j = 1; j < n; ++j) s = __fadd_rn(s, src[(int64_t)j * stride]);
  return s;
}

// Thread i < n_vec owns the 8-float slice i; the threads after them own one element each of the ragged tail.
// blockIdx.y selects the buffer (parameters, momentum).
__global__ void __launch_bounds__(kThreads)
partial_sum_kernel(const float* __restrict__ base, int64_t buf_stride, int m, int64_t n, int64_t stride,
                   float* __restrict__ out, int64_t out_stride) {
  grid_dep_wait();
  grid_dep_launch();
  const int64_t n_vec = n / 8;
  const int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x;
  const float* src = base + (int64_t)blockIdx.y * buf_stride;
  float* dst = out + (int64_t)blockIdx.y * out_stride;
  if (i < n_vec) {
    ordered_sum(src + i * 8, m, stride).store(dst + i * 8);
  } else {
    const int64_t e = n_vec * 8 + (i - n_vec);
    if (e < n) dst[e] = ordered_sum_scalar(src + e, m, stride);
  }
}

// parts: G vectors per buffer, vector g of buffer b at parts + g * part_stride + b * part_buf_stride
__global__ void __launch_bounds__(kThreads)
combine_kernel(const float* __restrict__ parts, int G, int64_t part_stride, int64_t part_buf_stride, float m_total,
               int64_t n, float* __restrict__ base, int64_t buf_stride, int m_local, int64_t stride,
               __nv_bfloat16* __restrict__ shadow, TileMap tiles) {
  grid_dep_wait();
  grid_dep_launch();
  const int64_t n_vec = n / 8;
  const int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x;
  const float* src = parts + (int64_t)blockIdx.y * part_buf_stride;
  float* dst = base + (int64_t)blockIdx.y * buf_stride;
  if (i < n_vec) {
    V8 s = ordered_sum(src + i * 8, G, part_stride);
#pragma unroll
    for (int e = 0; e < 8; ++e) s.v[e] = __fdiv_rn(s.v[e], m_total);
    for (int j = 0; j < m_local; ++j) s.store(dst + (int64_t)j * stride + i * 8);
    if (blockIdx.y == 0 && shadow != nullptr) {
      uint32_t u[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        __nv_bfloat162 t = __floats2bfloat162_rn(s.v[2 * e], s.v[2 * e + 1]);
        u[e] = *reinterpret_cast<uint32_t*>(&t);
      }
      const int64_t at = shadow_index(tiles, i * 8);
      for (int j = 0; j < m_local; ++j)
        *reinterpret_cast<uint4*>(shadow + (int64_t)j * stride + at) = make_uint4(u[0], u[1], u[2], u[3]);
    }
  } else {
    const int64_t e = n_vec * 8 + (i - n_vec);
    if (e < n) {
      const float mean = __fdiv_rn(ordered_sum_scalar(src + e, G, part_stride), m_total);
      for (int j = 0; j < m_local; ++j) dst[(int64_t)j * stride + e] = mean;
      if (blockIdx.y == 0 && shadow != nullptr) {
        const int64_t at = shadow_index(tiles, e);
        for (int j = 0; j < m_local; ++j) shadow[(int64_t)j * stride + at] = __float2bfloat16_rn(mean);
      }
    }
  }
}

inline bool aligned32(const void* p) { return reinterpret_cast<uintptr_t>(p) % 32 == 0; }
inline unsigned grid_x(int64_t n) { return (unsigned)((n / 8 + n % 8 + kThreads - 1) / kThreads); }

}  // namespace

int launch_partial_sum(const float* base, int n_buf, int64_t buf_stride, int m, int64_t n, int64_t stride, float* out,
                       int64_t out_stride, cudaStream_t st, int64_t* launches) {
  if (n <= 0 || n_buf <= 0) return cudaSuccess;
  if (!aligned32(base) || !aligned32(out) || stride % 8 != 0 || buf_stride % 8 != 0 || out_stride % 8 != 0 ||
      n / 8 + 8 > 2147483647LL * kThreads)
    return cudaErrorInvalidValue;
  if (launches) ++*launches;
  return launch_dep(partial_sum_kernel, dim3(grid_x(n), (unsigned)n_buf), dim3(kThreads), 0, st, 1, base, buf_stride, m,
                    n, stride, out, out_stride);
}

int launch_combine(const float* parts, int G, int64_t part_stride, int64_t part_buf_stride, int m_total, int64_t n,
                   float* base, int n_buf, int64_t buf_stride, int m_local, int64_t stride, __nv_bfloat16* shadow,
                   cudaStream_t st, int64_t* launches, const TileMap* tiles) {
  if (n <= 0 || n_buf <= 0) return cudaSuccess;
  if (!aligned32(parts) || !aligned32(base) || stride % 8 != 0 || buf_stride % 8 != 0 || part_stride % 8 != 0 ||
      part_buf_stride % 8 != 0 || reinterpret_cast<uintptr_t>(shadow) % 16 != 0 ||
      n / 8 + 8 > 2147483647LL * kThreads)
    return cudaErrorInvalidValue;
  if (launches) ++*launches;
  return launch_dep(combine_kernel, dim3(grid_x(n), (unsigned)n_buf), dim3(kThreads), 0, st, 1, parts, G, part_stride,
                    part_buf_stride, (float)m_total, n, base, buf_stride, m_local, stride, shadow,
                    tiles ? *tiles : TileMap{});
}

}  // namespace ls

extern "C" int ls_partial_sum_flat(const float* buf_dev, int m, int64_t P, int64_t stride, float* out_dev,
                                   void* cuda_stream) {
  if (buf_dev == nullptr || out_dev == nullptr || m < 1 || P < 0 || stride < P) return LS_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(buf_dev) % 32 != 0 || reinterpret_cast<uintptr_t>(out_dev) % 32 != 0 || stride % 8 != 0)
    return LS_ERR_INVALID_ARG;
  int e = ls::launch_partial_sum(buf_dev, 1, 0, m, P, stride, out_dev, 0, static_cast<cudaStream_t>(cuda_stream), nullptr);
  return e == cudaSuccess ? LS_OK : LS_ERR_CUDA;
}

extern "C" int ls_combine_partials_flat(const float* partials_dev, int G, int64_t part_stride, int m_total, int64_t P,
                                        float* dst_dev, int m_local, int64_t dst_stride, void* cuda_stream) {
  if (partials_dev == nullptr || dst_dev == nullptr || G < 1 || m_local < 1 || m_total < m_local || P < 0 ||
      part_stride < P || dst_stride < P)
    return LS_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(partials_dev) % 32 != 0 || reinterpret_cast<uintptr_t>(dst_dev) % 32 != 0 ||
      part_stride % 8 != 0 || dst_stride % 8 != 0)
    return LS_ERR_INVALID_ARG;
  int e = ls::launch_combine(partials_dev, G, part_stride, 0, m_total, P, dst_dev, 1, 0, m_local, dst_stride, nullptr,
                             static_cast<cudaStream_t>(cuda_stream), nullptr, nullptr);
  return e == cudaSuccess ? LS_OK : LS_ERR_CUDA;
}
