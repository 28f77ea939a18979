// The output layer when it is narrow (at most 16 outputs: the 10-class loss layer, or the
// single output of least squares).  Such a layer cannot fill a tensor-core tile, and as five
// generic launches (product, loss, two gradients, bias) it is all overhead, so it is two kernels:
//
//   head_fwd_kernel   z = A W^T + b, per-sample loss f(x; s_i), the mini-batch mean of it (the
//                     empirical risk of Section 2 restricted to the batch) and dZ = d(mean loss)/dz.
//                     Rows are spread over CTAs; the last CTA of a replica to finish adds the row
//                     losses in row order, so the mean does not depend on scheduling.
//   head_bwd_kernel   one pass over the layer input A for both gradients:
//                       dZ_prev = (dZ W) * 1[A > 0]          (skipped for a one-layer model)
//                       G = dZ^T A ; v <- mu v + G ; W <- W - eta v ; same for the bias
//                     (Section 2 mini-batch SGD update, Section 5.3 momentum).
//
// All sums run in a fixed order; W is read from the fp32 master copy.
#include "ls_internal.h"

namespace ls {
namespace {

constexpr int CMAX = 16;
constexpr int kThreads = 256;
constexpr int kRowsPerCta = 4;         // head_fwd: rows per CTA (the 8 warps split K)
constexpr int kColsPerCta = 64;        // head_bwd: 32 lanes x 2 columns, 8 row slices

__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ void put(float* p, float v) { *p = v; }
__device__ __forceinline__ void put(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

__device__ __forceinline__ void load4(const float* p, float (&r)[4]) {
  const float4 v = *reinterpret_cast<const float4*>(p);
  r[0] = v.x; r[1] = v.y; r[2] = v.z; r[3] = v.w;
}
__device__ __forceinline__ void load4(const __nv_bfloat16* p, float (&r)[4]) {
  uint2 u = *reinterpret_cast<const uint2*>(p);
  __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162*>(&u.x);
  __nv_bfloat162 b = *reinterpret_cast<__nv_bfloat162*>(&u.y);
  r[0] = __low2float(a); r[1] = __high2float(a); r[2] = __low2float(b); r[3] = __high2float(b);
}

// One CTA = kRowsPerCta (4) mini-batch rows of one replica.  The 8 warps split K; partial dot products are
// combined lane-wise by a butterfly and warp-wise through shared memory in warp order.
template <typename TA>
__global__ void __launch_bounds__(kThreads, 2)
head_fwd_kernel(const TA* __restrict__ A, const int64_t* __restrict__ a_row_off, const float* __restrict__ W,
                int64_t w_gstride, const float* __restrict__ bias, const void* __restrict__ y,
                const int64_t* __restrict__ y_row_off, float* __restrict__ dZ, float* __restrict__ row_loss,
                float* __restrict__ loss_out, unsigned int* __restrict__ counters, int B, int C, int K, int kind,
                int vec_ok) {
  __shared__ float part[8][kRowsPerCta * CMAX];
  __shared__ float zs[kRowsPerCta][CMAX];
  __shared__ unsigned int is_last;
  __shared__ float red[kThreads];
  grid_dep_wait();
  grid_dep_launch();
  const int g = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const TA* Ag = A + (a_row_off ? a_row_off[g] : (int64_t)g * B) * K;
  const float* Wg = W + (int64_t)g * w_gstride;
  const int b0 = blockIdx.x * kRowsPerCta;
  const int kchunk = (((K + 7) / 8) + 3) / 4 * 4;
  const int kw0 = warp * kchunk, kw1 = min(K, kw0 + kchunk);

  float acc[kRowsPerCta][CMAX];
#pragma unroll
  for (int r = 0; r < kRowsPerCta; ++r)
#pragma unroll
    for (int c = 0; c < CMAX; ++c) acc[r][c] = 0.f;
  if (vec_ok) {
    for (int k = kw0 + lane * 4; k < kw1; k += 128) {
      float a[kRowsPerCta][4];
#pragma unroll
      for (int r = 0; r < kRowsPerCta; ++r) {
        if (b0 + r < B) load4(Ag + (int64_t)(b0 + r) * K + k, a[r]);
        else a[r][0] = a[r][1] = a[r][2] = a[r][3] = 0.f;
      }
#pragma unroll
      for (int c = 0; c < CMAX; ++c)
        if (c < C) {
          float w[4];
          load4(Wg + (int64_t)c * K + k, w);
#pragma unroll
          for (int r = 0; r < kRowsPerCta; ++r)
            acc[r][c] = fmaf(a[r][3], w[3], fmaf(a[r][2], w[2], fmaf(a[r][1], w[1], fmaf(a[r][0], w[0], acc[r][c]))));
        }
    }
  } else {
    for (int k = kw0 + lane; k < kw1; k += 32) {
      float a[kRowsPerCta];
#pragma unroll
      for (int r = 0; r < kRowsPerCta; ++r) a[r] = (b0 + r < B) ? to_f(Ag[(int64_t)(b0 + r) * K + k]) : 0.f;
#pragma unroll
      for (int c = 0; c < CMAX; ++c)
        if (c < C) {
          const float w = Wg[(int64_t)c * K + k];
#pragma unroll
          for (int r = 0; r < kRowsPerCta; ++r) acc[r][c] = fmaf(a[r], w, acc[r][c]);
        }
    }
  }
#pragma unroll
  for (int r = 0; r < kRowsPerCta; ++r)
#pragma unroll
    for (int c = 0; c < CMAX; ++c)
      if (c < C) {
        float v = acc[r][c];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0) part[warp][r * CMAX + c] = v;
      }
  __syncthreads();
  if (threadIdx.x < kRowsPerCta * CMAX) {
    const int r = threadIdx.x / CMAX, c = threadIdx.x % CMAX;
    float s = 0.f;
    if (c < C) {
#pragma unroll
      for (int w = 0; w < 8; ++w) s += part[w][threadIdx.x];
      if (bias) s += bias[(int64_t)g * w_gstride + c];
    }
    zs[r][c] = s;
  }
  __syncthreads();
  const float invB = 1.0f / (float)B;
  if (warp < kRowsPerCta && b0 + warp < B) {
    // warp r finishes row r: lane c holds class c
    const int b = b0 + warp;
    const int64_t y0 = y_row_off[g];
    const float z = (lane < C) ? zs[warp][lane] : -INFINITY;
    float loss, d;
    if (kind == LS_LOSS_SOFTMAX_CE) {
      const int label = static_cast<const int32_t*>(y)[y0 + b];
      float mx = z;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      const float e = (lane < C) ? expf(z - mx) : 0.f;
      float sum = e;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      const float zy = __shfl_sync(0xffffffffu, z, (label >= 0 && label < C) ? label : 0);
      loss = (mx + logf(sum)) - ((label >= 0 && label < C) ? zy : mx);
      d = (e / sum - (lane == label ? 1.f : 0.f)) * invB;
    } else {
      const float res = zs[warp][0] - static_cast<const float*>(y)[y0 + b];
      loss = 0.5f * res * res;
      d = res * invB;
    }
    if (lane == 0) row_loss[(int64_t)g * B + b] = loss;
    if (dZ != nullptr && lane < C) dZ[((int64_t)g * B + b) * C + lane] = d;
  }
  // the last CTA of this replica adds the row losses in row order
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) is_last = (atomicInc(&counters[g], gridDim.x - 1) == gridDim.x - 1) ? 1u : 0u;
  __syncthreads();
  if (is_last && loss_out != nullptr) {
    __threadfence();
    float p = 0.f;
    for (int b = threadIdx.x; b < B; b += kThreads) p += __ldcg(&row_loss[(int64_t)g * B + b]);
    red[threadIdx.x] = p;
    __syncthreads();
    for (int s = kThreads / 2; s > 0; s >>= 1) {
      if (threadIdx.x < s) red[threadIdx.x] += red[threadIdx.x + s];
      __syncthreads();
    }
    if (threadIdx.x == 0) loss_out[g] = red[0] * invB;
  }
}

__device__ __forceinline__ void load2(const float* p, float (&r)[2]) {
  const float2 v = *reinterpret_cast<const float2*>(p);
  r[0] = v.x; r[1] = v.y;
}
__device__ __forceinline__ void load2(const __nv_bfloat16* p, float (&r)[2]) {
  const __nv_bfloat162 v = *reinterpret_cast<const __nv_bfloat162*>(p);
  r[0] = __low2float(v); r[1] = __high2float(v);
}
__device__ __forceinline__ void store2(float* p, float a, float b) { *reinterpret_cast<float2*>(p) = make_float2(a, b); }
__device__ __forceinline__ void store2(__nv_bfloat16* p, float a, float b) {
  *reinterpret_cast<__nv_bfloat162*>(p) = __floats2bfloat162_rn(a, b);
}

// One CTA = kColsPerCta (64) columns of the layer input of one replica: 32 lanes x 2 adjacent columns,
// 8 warps = 8 interleaved row slices.  pair_ok: K is even and the pointers are aligned for 2-element accesses.
template <typename TA>
__global__ void __launch_bounds__(kThreads, 2)
head_bwd_kernel(const TA* __restrict__ A, const int64_t* __restrict__ a_row_off, const float* __restrict__ dZ,
                float* __restrict__ W, float* __restrict__ V, __nv_bfloat16* __restrict__ Wb,
                float* __restrict__ bias, float* __restrict__ vbias, int64_t w_gstride, TA* __restrict__ dPrev,
                float* __restrict__ pbias, float* __restrict__ pvbias, int B, int C, int K, float lr, float mu,
                int pair_ok) {
  extern __shared__ float sm[];
  float* dz = sm;                                   // [B][C]
  float* part = sm + (size_t)B * C;                 // [8][CMAX][kColsPerCta]
  grid_dep_wait();
  grid_dep_launch();
  const int g = blockIdx.y;
  const int cx = threadIdx.x & 31, ry = threadIdx.x >> 5;
  const int k = blockIdx.x * kColsPerCta + cx * 2;  // this thread's columns k, k + 1
  const TA* Ag = A + (a_row_off ? a_row_off[g] : (int64_t)g * B) * K;
  const bool in0 = k < K, in1 = k + 1 < K;

  float wreg[CMAX][2], gw[CMAX][2];
#pragma unroll
  for (int c = 0; c < CMAX; ++c) {
    wreg[c][0] = (c < C && in0) ? W[(int64_t)g * w_gstride + (int64_t)c * K + k] : 0.f;
    wreg[c][1] = (c < C && in1) ? W[(int64_t)g * w_gstride + (int64_t)c * K + k + 1] : 0.f;
    gw[c][0] = gw[c][1] = 0.f;
  }
  float cs0 = 0.f, cs1 = 0.f;     // column sums of dPrev over this thread's rows (bias gradient of the layer below)
  for (int i = threadIdx.x; i < B * C; i += kThreads) dz[i] = dZ[(int64_t)g * B * C + i];
  __syncthreads();

  if (in0) {
    for (int bb = ry; bb < B; bb += 64) {
      // eight rows per trip so that eight loads of A are in flight
      float av[8][2];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        av[u][0] = av[u][1] = 0.f;
        if (bb + 8 * u < B) {
          const TA* src = Ag + (int64_t)(bb + 8 * u) * K + k;
          if (pair_ok) load2(src, av[u]);
          else { av[u][0] = to_f(src[0]); if (in1) av[u][1] = to_f(src[1]); }
        }
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int b = bb + 8 * u;
        if (b >= B) break;
        float da0 = 0.f, da1 = 0.f;
#pragma unroll
        for (int c = 0; c < CMAX; ++c)
          if (c < C) {
            const float d = dz[b * C + c];
            gw[c][0] = fmaf(d, av[u][0], gw[c][0]);
            gw[c][1] = fmaf(d, av[u][1], gw[c][1]);
            da0 = fmaf(d, wreg[c][0], da0);
            da1 = fmaf(d, wreg[c][1], da1);
          }
        if (dPrev != nullptr) {
          const float o0 = av[u][0] > 0.f ? da0 : 0.f, o1 = av[u][1] > 0.f ? da1 : 0.f;
          cs0 += o0;
          cs1 += o1;
          const int64_t at = ((int64_t)g * B + b) * K + k;
          if (pair_ok) {
            store2(dPrev + at, o0, o1);
          } else {
            put(dPrev + at, o0);
            if (in1) put(dPrev + at + 1, o1);
          }
        }
      }
    }
  }
#pragma unroll
  for (int c = 0; c < CMAX; ++c) {
    part[(ry * CMAX + c) * kColsPerCta + cx * 2] = gw[c][0];
    part[(ry * CMAX + c) * kColsPerCta + cx * 2 + 1] = gw[c][1];
  }
  __syncthreads();
  // 8 warps x 64 columns: thread t < 64 * C finishes column t % 64 of output row t / 64 ... done by all
  // threads in a strided loop so that the V / W accesses are coalesced along k
  for (int t = threadIdx.x; t < C * kColsPerCta; t += kThreads) {
    const int c = t / kColsPerCta, col = t % kColsPerCta;
    const int kk = blockIdx.x * kColsPerCta + col;
    if (kk >= K) continue;
    float s = 0.f;
#pragma unroll
    for (int r = 0; r < 8; ++r) s += part[(r * CMAX + c) * kColsPerCta + col];
    const int64_t at = (int64_t)g * w_gstride + (int64_t)c * K + kk;
    float step = s;
    if (mu != 0.f) {
      step = fmaf(mu, V[at], s);
      V[at] = step;
    }
    const float w = fmaf(-lr, step, W[at]);
    W[at] = w;
    if (Wb != nullptr) Wb[at] = __float2bfloat16_rn(w);
  }
  if (blockIdx.x == 0 && bias != nullptr && threadIdx.x < C) {
    const int c = threadIdx.x;
    float s = 0.f;
    for (int b = 0; b < B; ++b) s += dz[b * C + c];
    const int64_t at = (int64_t)g * w_gstride + c;
    float step = s;
    if (mu != 0.f) {
      step = fmaf(mu, vbias[at], s);
      vbias[at] = step;
    }
    bias[at] = fmaf(-lr, step, bias[at]);
  }
  if (pbias != nullptr) {
    // bias of the layer below: its gradient is the column sum of dPrev, complete inside this CTA
    __syncthreads();
    part[ry * kColsPerCta + cx * 2] = cs0;
    part[ry * kColsPerCta + cx * 2 + 1] = cs1;
    __syncthreads();
    const int kk = blockIdx.x * kColsPerCta + threadIdx.x;
    if (threadIdx.x < kColsPerCta && kk < K) {
      float s = 0.f;
#pragma unroll
      for (int r = 0; r < 8; ++r) s += part[r * kColsPerCta + threadIdx.x];
      const int64_t at = (int64_t)g * w_gstride + kk;
      float step = s;
      if (mu != 0.f) {
        step = fmaf(mu, pvbias[at], s);
        pvbias[at] = step;
      }
      pbias[at] = fmaf(-lr, step, pbias[at]);
    }
  }
}

}  // namespace

bool head_shape_ok(int B, int C) { return C >= 1 && C <= CMAX && B >= 1 && (size_t)B * C * 4 <= 64 * 1024; }

int launch_head_fwd(const HeadFwdArgs& a, bool a_bf16, cudaStream_t st, int64_t* launches) {
  if (launches) ++*launches;
  dim3 grid((unsigned)((a.B + kRowsPerCta - 1) / kRowsPerCta), (unsigned)a.groups);
  const int vec_ok = (a.K % 4 == 0) && (reinterpret_cast<uintptr_t>(a.A) % 16 == 0) &&
                     (reinterpret_cast<uintptr_t>(a.W) % 16 == 0) && (a.w_gstride % 4 == 0);
  if (a_bf16)
    return launch_dep(head_fwd_kernel<__nv_bfloat16>, grid, dim3(kThreads), 0, st, 1,
                      static_cast<const __nv_bfloat16*>(a.A), a.a_row_off, a.W, a.w_gstride, a.bias, a.y, a.y_row_off,
                      a.dZ, a.row_loss, a.loss_out, a.counters, a.B, a.C, a.K, a.loss_kind, vec_ok);
  return launch_dep(head_fwd_kernel<float>, grid, dim3(kThreads), 0, st, 1, static_cast<const float*>(a.A),
                    a.a_row_off, a.W, a.w_gstride, a.bias, a.y, a.y_row_off, a.dZ, a.row_loss, a.loss_out, a.counters,
                    a.B, a.C, a.K, a.loss_kind, vec_ok);
}

int launch_head_bwd(const HeadBwdArgs& a, bool a_bf16, cudaStream_t st, int64_t* launches) {
  if (launches) ++*launches;
  dim3 grid((unsigned)((a.K + kColsPerCta - 1) / kColsPerCta), (unsigned)a.groups);
  const size_t smem = ((size_t)a.B * a.C + 8 * CMAX * kColsPerCta) * sizeof(float);
  const size_t esz = a_bf16 ? 2 : 4;
  const int pair_ok = (a.K % 2 == 0) && reinterpret_cast<uintptr_t>(a.A) % (2 * esz) == 0 &&
                      (a.dPrev == nullptr || reinterpret_cast<uintptr_t>(a.dPrev) % (2 * esz) == 0);
  if (a_bf16) {
    auto kern = head_bwd_kernel<__nv_bfloat16>;
    static bool configured = false;
    if (!configured) {
      cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024);
      if (e != cudaSuccess) return e;
      configured = true;
    }
    return launch_dep(kern, grid, dim3(kThreads), smem, st, 1, static_cast<const __nv_bfloat16*>(a.A), a.a_row_off,
                      a.dZ, a.W, a.V, a.Wb, a.bias, a.vbias, a.w_gstride, static_cast<__nv_bfloat16*>(a.dPrev),
                      a.dPrev ? a.pbias : nullptr, a.pvbias, a.B, a.C, a.K, a.lr, a.mu, pair_ok);
  } else {
    auto kern = head_bwd_kernel<float>;
    static bool configured = false;
    if (!configured) {
      cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024);
      if (e != cudaSuccess) return e;
      configured = true;
    }
    return launch_dep(kern, grid, dim3(kThreads), smem, st, 1, static_cast<const float*>(a.A), a.a_row_off, a.dZ,
                      a.W, a.V, a.Wb, a.bias, a.vbias, a.w_gstride, static_cast<float*>(a.dPrev),
                      a.dPrev ? a.pbias : nullptr, a.pvbias, a.B, a.C, a.K, a.lr, a.mu, pair_ok);
  }
}

}  // namespace ls

// ---------------------------------------------------------------------------
// ls_linear_loss_static: the output-layer kernel for callers that cannot allocate.
// ---------------------------------------------------------------------------
namespace {

constexpr int kStaticMaxChunks = 256;       // chunks (groups) per call
constexpr int kStaticMaxRows = 65536;       // rows per call
// Scratch of the kernel: CTA counters, per-chunk first rows, per-row losses.  It lives in the
// library image, so every GPU that loads the library holds these ~260 KB until the process exits.
struct StaticScratch {
  unsigned int counters[kStaticMaxChunks];
  long long row_off[kStaticMaxChunks];
  float row_loss[kStaticMaxRows];
};
static __device__ __align__(256) unsigned char g_static_scratch[sizeof(StaticScratch)];

// Device address of the scratch, looked up once per device (index = CUDA device ordinal).
static StaticScratch* g_scratch_addr[64] = {nullptr};

}  // namespace

extern "C" int ls_linear_loss_static(const float* W_dev, const float* bias_dev, const float* x_dev, const void* y_dev,
                                     int64_t n_rows, int d_in, int d_out, int loss, int chunk_rows,
                                     float* chunk_loss_dev, void* cuda_stream) {
  using namespace ls;
  if (W_dev == nullptr || x_dev == nullptr || y_dev == nullptr || chunk_loss_dev == nullptr) return LS_ERR_INVALID_ARG;
  if (d_in < 1 || d_out < 1 || chunk_rows < 1 || n_rows < chunk_rows || n_rows % chunk_rows != 0)
    return LS_ERR_INVALID_ARG;
  if (loss != LS_LOSS_SOFTMAX_CE && loss != LS_LOSS_MSE_HALF) return LS_ERR_INVALID_ARG;
  if (loss == LS_LOSS_MSE_HALF && d_out != 1) return LS_ERR_INVALID_ARG;
  const int64_t chunks = n_rows / chunk_rows;
  if (d_out > CMAX || chunks > kStaticMaxChunks || n_rows > kStaticMaxRows || chunk_rows > LS_MAX_BATCH)
    return LS_ERR_TOO_LARGE;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return LS_ERR_CUDA;
  if (g_scratch_addr[dev] == nullptr) {
    // In host code the array's name is only a handle: ask the runtime for its address on this device.
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return LS_ERR_CUDA;
    g_scratch_addr[dev] = static_cast<StaticScratch*>(p);
  }
  StaticScratch* sc = g_scratch_addr[dev];
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  // the counters must start at zero; the first row of every chunk is chunk * chunk_rows
  if (cudaMemsetAsync(sc->counters, 0, sizeof(sc->counters), st) != cudaSuccess) return LS_ERR_CUDA;
  long long offs[kStaticMaxChunks];
  for (int64_t c = 0; c < chunks; ++c) offs[c] = c * (long long)chunk_rows;
  if (cudaMemcpyAsync(sc->row_off, offs, (size_t)chunks * sizeof(long long), cudaMemcpyHostToDevice, st) != cudaSuccess)
    return LS_ERR_CUDA;
  HeadFwdArgs a;
  a.A = x_dev; a.a_row_off = reinterpret_cast<const int64_t*>(sc->row_off);
  a.W = W_dev; a.w_gstride = 0; a.bias = bias_dev;
  a.y = y_dev; a.y_row_off = reinterpret_cast<const int64_t*>(sc->row_off);
  a.dZ = nullptr;
  a.row_loss = sc->row_loss; a.loss_out = chunk_loss_dev; a.counters = sc->counters;
  a.B = chunk_rows; a.C = d_out; a.K = d_in; a.groups = (int)chunks; a.loss_kind = loss;
  return launch_head_fwd(a, false, st, nullptr) == cudaSuccess ? LS_OK : LS_ERR_CUDA;
}
