// Loss layer and small per-layer kernels.
//
//   loss_kernel   per-sample loss f(x; s_i), its mini-batch mean (the
//                 empirical risk of Section 2 restricted to the batch) and the
//                 gradient of that mean with respect to the network output:
//                   softmax cross-entropy  dZ = (softmax(z) - onehot(y)) / |xi|
//                   half squared error     dZ = (z - y) / |xi|
//   bias_kernel   gb = column sums of dZ; v <- mu v + gb; b <- b - eta v
//   to_bf16       refresh of the bf16 weight copies
//
// All sums run in a fixed order (no floating-point atomics).
#include "ls_internal.h"

namespace ls {
namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ void put(float* p, float v) { *p = v; }
__device__ __forceinline__ void put(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

template <typename TD>
__global__ void __launch_bounds__(kThreads)
loss_kernel(const float* __restrict__ logits, const void* __restrict__ y, const int64_t* __restrict__ row_off,
            TD* __restrict__ dZ, float* __restrict__ loss_out, int B, int C, int kind) {
  __shared__ float red[kThreads];
  grid_dep_wait();
  grid_dep_launch();
  const int g = blockIdx.x;
  const float* z = logits + (int64_t)g * B * C;
  TD* dz = dZ ? dZ + (int64_t)g * B * C : nullptr;
  const int64_t r0 = row_off[g];
  const float invB = 1.0f / (float)B;
  float part = 0.f;
  for (int b = threadIdx.x; b < B; b += kThreads) {
    const float* zb = z + (int64_t)b * C;
    if (kind == LS_LOSS_SOFTMAX_CE) {
      const int label = static_cast<const int32_t*>(y)[r0 + b];
      float mx = zb[0];
      for (int c = 1; c < C; ++c) mx = fmaxf(mx, zb[c]);
      float sum = 0.f;
      for (int c = 0; c < C; ++c) sum += expf(zb[c] - mx);
      const float zy = (label >= 0 && label < C) ? zb[label] : mx;
      part += (mx + logf(sum)) - zy;
      if (dz) {
        const float inv = 1.0f / sum;
        for (int c = 0; c < C; ++c) {
          const float p = expf(zb[c] - mx) * inv;
          const float d = (p - (c == label ? 1.f : 0.f)) * invB;
          put(dz + (int64_t)b * C + c, d);
        }
      }
    } else {
      const float t = static_cast<const float*>(y)[r0 + b];
      const float r = zb[0] - t;
      part += 0.5f * r * r;
      if (dz) put(dz + b, r * invB);
    }
  }
  red[threadIdx.x] = part;
  __syncthreads();
  for (int s = kThreads / 2; s > 0; s >>= 1) {
    if (threadIdx.x < s) red[threadIdx.x] += red[threadIdx.x + s];
    __syncthreads();
  }
  if (threadIdx.x == 0 && loss_out) loss_out[g] = red[0] * invB;
}

template <typename TD>
__global__ void __launch_bounds__(kThreads)
bias_kernel(const TD* __restrict__ dZ, float* __restrict__ bias, float* __restrict__ vbias, int64_t gstride, int B,
            int N, float lr, float mu) {
  // 32 columns x 8 row slices per block: each thread adds every 8th row, then the 8 partial sums of a
  // column are added in slice order
  __shared__ float part[8][32];
  grid_dep_wait();
  grid_dep_launch();
  const int g = blockIdx.y;
  const int cx = threadIdx.x & 31, ry = threadIdx.x >> 5;
  const int j = blockIdx.x * 32 + cx;
  float s = 0.f;
  if (j < N) {
    const TD* d = dZ + (int64_t)g * B * N + j;
    for (int b = ry; b < B; b += 8) {
      if constexpr (sizeof(TD) == 2) s += __bfloat162float(d[(int64_t)b * N]);
      else s += d[(int64_t)b * N];
    }
  }
  part[ry][cx] = s;
  __syncthreads();
  if (ry != 0 || j >= N) return;
  s = 0.f;
#pragma unroll
  for (int r = 0; r < 8; ++r) s += part[r][cx];
  const int64_t at = (int64_t)g * gstride + j;
  float step = s;
  if (mu != 0.f) {
    step = fmaf(mu, vbias[at], s);
    vbias[at] = step;
  }
  bias[at] = fmaf(-lr, step, bias[at]);
}

// eight consecutive elements per thread (replica vectors are padded to multiples of 64): one index translation
// and one 16-byte store for each
__global__ void __launch_bounds__(kThreads)
to_bf16_kernel(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst, int64_t stride, int64_t n, TileMap tiles) {
  const int64_t step = (int64_t)gridDim.x * kThreads;
  for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < n / 8; i += step) {
    const int64_t e0 = i * 8, rep = e0 / stride, e = e0 - rep * stride;
    const float4 a = *reinterpret_cast<const float4*>(src + e0), b = *reinterpret_cast<const float4*>(src + e0 + 4);
    __nv_bfloat162 p0 = __floats2bfloat162_rn(a.x, a.y), p1 = __floats2bfloat162_rn(a.z, a.w);
    __nv_bfloat162 p2 = __floats2bfloat162_rn(b.x, b.y), p3 = __floats2bfloat162_rn(b.z, b.w);
    *reinterpret_cast<uint4*>(dst + rep * stride + shadow_index(tiles, e)) =
        make_uint4(*reinterpret_cast<uint32_t*>(&p0), *reinterpret_cast<uint32_t*>(&p1), *reinterpret_cast<uint32_t*>(&p2),
                   *reinterpret_cast<uint32_t*>(&p3));
  }
}

// one CTA per 32 x 32 block; a warp moves one 128-byte row at a time on both sides
__global__ void __launch_bounds__(kThreads)
retile_kernel(float* __restrict__ dst, const float* __restrict__ src, int rows, int cols, int to_blocked) {
  const int nb = cols >> 5;
  const int64_t blk = blockIdx.x;
  const int rb = (int)(blk / nb), cb = (int)(blk % nb);
  const int c = threadIdx.x & 31, r0 = threadIdx.x >> 5;
  for (int r = r0; r < 32; r += kThreads / 32) {
    const int64_t rm = (int64_t)(rb * 32 + r) * cols + cb * 32 + c, bl = blk * 1024 + r * 32 + c;
    if (to_blocked) dst[bl] = src[rm];
    else dst[rm] = src[bl];
  }
}

}  // namespace

int launch_loss(const LossArgs& a, bool dz_bf16, cudaStream_t st, int64_t* launches) {
  if (launches) ++*launches;
  if (dz_bf16)
    return launch_dep(loss_kernel<__nv_bfloat16>, dim3(a.groups), dim3(kThreads), 0, st, 1, a.logits, a.y, a.row_off,
                      static_cast<__nv_bfloat16*>(a.dZ), a.loss_out, a.B, a.C, a.loss_kind);
  return launch_dep(loss_kernel<float>, dim3(a.groups), dim3(kThreads), 0, st, 1, a.logits, a.y, a.row_off,
                    static_cast<float*>(a.dZ), a.loss_out, a.B, a.C, a.loss_kind);
}

int launch_bias(const BiasArgs& a, bool bf16, cudaStream_t st, int64_t* launches) {
  if (launches) ++*launches;
  dim3 grid((unsigned)((a.N + 31) / 32), (unsigned)a.groups);
  if (bf16)
    return launch_dep(bias_kernel<__nv_bfloat16>, grid, dim3(kThreads), 0, st, 1,
                      static_cast<const __nv_bfloat16*>(a.dZ), a.bias, a.vbias, a.gstride, a.B, a.N, a.lr, a.mu);
  return launch_dep(bias_kernel<float>, grid, dim3(kThreads), 0, st, 1, static_cast<const float*>(a.dZ), a.bias,
                    a.vbias, a.gstride, a.B, a.N, a.lr, a.mu);
}

int launch_to_bf16(const float* src, __nv_bfloat16* dst, int m, int64_t stride, const TileMap* tiles, cudaStream_t st,
                   int64_t* launches) {
  const int64_t n = (int64_t)m * stride;
  if (n <= 0) return cudaSuccess;
  if (launches) ++*launches;
  if (stride % 8 != 0 || reinterpret_cast<uintptr_t>(src) % 16 != 0 || reinterpret_cast<uintptr_t>(dst) % 16 != 0)
    return cudaErrorInvalidValue;
  int64_t gx = (n / 8 + kThreads - 1) / kThreads;
  if (gx > 148 * 16) gx = 148 * 16;
  to_bf16_kernel<<<(unsigned)gx, kThreads, 0, st>>>(src, dst, stride, n, tiles ? *tiles : TileMap{});
  return cudaGetLastError();
}

int launch_retile(float* dst, const float* src, int rows, int cols, bool to_blocked, cudaStream_t st, int64_t* launches) {
  if (rows <= 0 || cols <= 0 || rows % 32 != 0 || cols % 32 != 0) return cudaErrorInvalidValue;
  if (launches) ++*launches;
  retile_kernel<<<(unsigned)((int64_t)rows * cols / 1024), kThreads, 0, st>>>(dst, src, rows, cols, to_blocked ? 1 : 0);
  return cudaGetLastError();
}

}  // namespace ls
