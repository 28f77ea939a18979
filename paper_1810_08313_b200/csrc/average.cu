// Model averaging: X <- X J, J = 1 1^T / m (Section 2, PASGD update rule, the
// case k mod tau = 0; operator J of the convergence proof's notation).
//
// Bandwidth-bound streaming kernel.  Every thread owns one 16-byte column
// slice: it issues the m independent 128-bit loads of that slice (one per
// replica) before using any of them, adds them in replica order in fp32,
// divides once by (float)m and stores the mean back to all m replicas.
// Algorithmic traffic is 8*m bytes per parameter: each element is read once
// and written once.  No shared memory, no inter-thread communication: the
// reduction order is fixed by construction, so the result is bit-reproducible.
#include "ls_internal.h"

namespace ls {

namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ float4 add4(float4 a, float4 b) {
  // plain IEEE adds; no multiply nearby, so nothing can be contracted into an FMA
  return make_float4(__fadd_rn(a.x, b.x), __fadd_rn(a.y, b.y), __fadd_rn(a.z, b.z), __fadd_rn(a.w, b.w));
}
__device__ __forceinline__ float4 div4(float4 a, float d) {
  return make_float4(__fdiv_rn(a.x, d), __fdiv_rn(a.y, d), __fdiv_rn(a.z, d), __fdiv_rn(a.w, d));
}
__device__ __forceinline__ float tf32_lo(float x) { return x - __uint_as_float(__float_as_uint(x) & 0xFFFFE000u); }
__device__ __forceinline__ void store_bf16x4(__nv_bfloat16* p, float4 v) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y);
  __nv_bfloat162 hi = __floats2bfloat162_rn(v.z, v.w);
  uint2 u;
  u.x = *reinterpret_cast<uint32_t*>(&lo);
  u.y = *reinterpret_cast<uint32_t*>(&hi);
  *reinterpret_cast<uint2*>(p) = u;
}

// M > 0: replica count known at compile time (loads fully unrolled, all in flight).
// M == 0: any m, processed in chunks of 8 loads, still in replica order.
template <int M>
__global__ void __launch_bounds__(kThreads)
average_vec4_kernel(float* __restrict__ base, int64_t buf_stride, int m_rt, int64_t n_vec, int64_t stride,
                    __nv_bfloat16* __restrict__ shadow, float* __restrict__ lo) {
  const int m = M > 0 ? M : m_rt;
  float* buf = base + (int64_t)blockIdx.y * buf_stride;
  const bool do_shadow = (shadow != nullptr) && blockIdx.y == 0;
  const bool do_lo = (lo != nullptr) && blockIdx.y == 0;
  const float mf = (float)m;
  const int64_t step = (int64_t)gridDim.x * kThreads;
  for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < n_vec; i += step) {
    float4* p = reinterpret_cast<float4*>(buf) + i;
    const int64_t s4 = stride / 4;
    float4 mean;
    if (M > 0) {
      float4 v[M > 0 ? M : 1];
#pragma unroll
      for (int j = 0; j < M; ++j) v[j] = __ldcs(p + j * s4);
      float4 s = v[0];
#pragma unroll
      for (int j = 1; j < M; ++j) s = add4(s, v[j]);
      mean = div4(s, mf);
    } else {
      float4 s = __ldcs(p);
      for (int j0 = 1; j0 < m; j0 += 8) {
        float4 v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (j0 + j < m) v[j] = __ldcs(p + (int64_t)(j0 + j) * s4);
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (j0 + j < m) s = add4(s, v[j]);
      }
      mean = div4(s, mf);
    }
#pragma unroll 4
    for (int j = 0; j < m; ++j) p[(int64_t)j * s4] = mean;
    if (do_shadow) {
      for (int j = 0; j < m; ++j) store_bf16x4(shadow + (int64_t)j * stride + i * 4, mean);
    }
    if (do_lo) {
      const float4 l4 = make_float4(tf32_lo(mean.x), tf32_lo(mean.y), tf32_lo(mean.z), tf32_lo(mean.w));
      for (int j = 0; j < m; ++j) *reinterpret_cast<float4*>(lo + (int64_t)j * stride + i * 4) = l4;
    }
  }
}

// Scalar path: the ragged tail (n mod 4 elements) and buffers that are not
// 16-byte aligned.  Same arithmetic, one element per thread.
__global__ void __launch_bounds__(kThreads)
average_scalar_kernel(float* __restrict__ base, int64_t buf_stride, int m, int64_t first, int64_t n, int64_t stride,
                      __nv_bfloat16* __restrict__ shadow, float* __restrict__ lo) {
  float* buf = base + (int64_t)blockIdx.y * buf_stride;
  const bool do_shadow = (shadow != nullptr) && blockIdx.y == 0;
  const float mf = (float)m;
  const int64_t step = (int64_t)gridDim.x * kThreads;
  for (int64_t i = first + (int64_t)blockIdx.x * kThreads + threadIdx.x; i < n; i += step) {
    float s = buf[i];
    for (int j = 1; j < m; ++j) s = __fadd_rn(s, buf[(int64_t)j * stride + i]);
    const float mean = __fdiv_rn(s, mf);
    for (int j = 0; j < m; ++j) buf[(int64_t)j * stride + i] = mean;
    if (do_shadow)
      for (int j = 0; j < m; ++j) shadow[(int64_t)j * stride + i] = __float2bfloat16_rn(mean);
    if (lo != nullptr && blockIdx.y == 0)
      for (int j = 0; j < m; ++j) lo[(int64_t)j * stride + i] = tf32_lo(mean);
  }
}

int num_sms() {
  static int sms = 0;
  if (sms == 0) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) sms = 148;
  }
  return sms;
}

template <int M>
void launch_vec4(dim3 grid, cudaStream_t st, float* base, int64_t buf_stride, int m, int64_t n_vec, int64_t stride,
                 __nv_bfloat16* shadow, float* lo) {
  average_vec4_kernel<M><<<grid, kThreads, 0, st>>>(base, buf_stride, m, n_vec, stride, shadow, lo);
}

}  // namespace

int launch_average(float* base, int n_buf, int64_t buf_stride, int m, int64_t n, int64_t stride,
                   __nv_bfloat16* shadow, float* lo, cudaStream_t st, int64_t* launches) {
  if (n <= 0 || n_buf <= 0) return cudaSuccess;
  const bool aligned = (reinterpret_cast<uintptr_t>(base) % 16 == 0) && (stride % 4 == 0) && (buf_stride % 4 == 0) &&
                       (shadow == nullptr || reinterpret_cast<uintptr_t>(shadow) % 8 == 0) &&
                       (lo == nullptr || reinterpret_cast<uintptr_t>(lo) % 16 == 0);
  const int64_t n_vec = aligned ? n / 4 : 0;
  const int sms = num_sms();
  if (n_vec > 0) {
    // whole multiples of the SM count; each thread keeps m 16-byte loads in flight
    int per_sm = m <= 8 ? 8 : 4;
    int64_t want = (n_vec + kThreads - 1) / kThreads;
    int64_t gx = (int64_t)sms * per_sm;
    if (want < gx) gx = want;
    dim3 grid((unsigned)gx, (unsigned)n_buf);
    switch (m) {
      case 2: launch_vec4<2>(grid, st, base, buf_stride, m, n_vec, stride, shadow, lo); break;
      case 4: launch_vec4<4>(grid, st, base, buf_stride, m, n_vec, stride, shadow, lo); break;
      case 8: launch_vec4<8>(grid, st, base, buf_stride, m, n_vec, stride, shadow, lo); break;
      case 16: launch_vec4<16>(grid, st, base, buf_stride, m, n_vec, stride, shadow, lo); break;
      default: launch_vec4<0>(grid, st, base, buf_stride, m, n_vec, stride, shadow, lo); break;
    }
    if (launches) ++*launches;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  const int64_t first = n_vec * 4;
  if (first < n) {
    int64_t rem = n - first;
    int64_t gx = (rem + kThreads - 1) / kThreads;
    if (gx > (int64_t)sms * 8) gx = (int64_t)sms * 8;
    dim3 grid((unsigned)gx, (unsigned)n_buf);
    average_scalar_kernel<<<grid, kThreads, 0, st>>>(base, buf_stride, m, first, n, stride, shadow, lo);
    if (launches) ++*launches;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace ls

extern "C" int ls_average_flat(float* buf_dev, int m, int64_t P, int64_t stride, void* cuda_stream) {
  if (buf_dev == nullptr || m < 1 || P < 0 || stride < P) return LS_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(buf_dev) % 4 != 0) return LS_ERR_INVALID_ARG;
  int e = ls::launch_average(buf_dev, 1, 0, m, P, stride, nullptr, nullptr, static_cast<cudaStream_t>(cuda_stream),
                             nullptr);
  return e == cudaSuccess ? LS_OK : LS_ERR_CUDA;
}
