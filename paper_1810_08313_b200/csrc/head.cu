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
// CT: the number of outputs when it is known at compile time (10 classes, 1 regression output), else 0.  With
// a run-time count the class loops need an early exit, and a load behind a branch cannot be issued before
// the branch: the loads of the classes then go out one round trip at a time.
template <typename TA, int CT>
__global__ void __launch_bounds__(kThreads, 2)
head_fwd_kernel(const TA* __restrict__ A, const int64_t* __restrict__ a_row_off, const float* __restrict__ W,
                int64_t w_gstride, const float* __restrict__ bias, const void* __restrict__ y,
                const int64_t* __restrict__ y_row_off, float* __restrict__ dZ, float* __restrict__ row_loss,
                float* __restrict__ loss_out, unsigned int* __restrict__ counters, int B, int C, int K, int kind,
                int vec_ok, int defer_loss) {
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
  // what the end of the kernel needs is requested now, so that it arrives with the operands:
  // the bias (thread (row, class)) and the label / target of row `warp`
  float bz = 0.f;
  if (bias != nullptr && threadIdx.x < kRowsPerCta * CMAX && (threadIdx.x % CMAX) < C)
    bz = bias[(int64_t)g * w_gstride + (threadIdx.x % CMAX)];
  int label = 0;
  float target = 0.f;
  if (warp < kRowsPerCta && b0 + warp < B) {
    const int64_t y0 = y_row_off[g];
    if (kind == LS_LOSS_SOFTMAX_CE) label = static_cast<const int32_t*>(y)[y0 + b0 + warp];
    else target = static_cast<const float*>(y)[y0 + b0 + warp];
  }

  constexpr int CU = CT > 0 ? CT : CMAX;      // unrolled class count
  float acc[kRowsPerCta][CU];
#pragma unroll
  for (int r = 0; r < kRowsPerCta; ++r)
#pragma unroll
    for (int c = 0; c < CU; ++c) acc[r][c] = 0.f;
  if (vec_ok) {
    for (int k = kw0 + lane * 4; k < kw1; k += 128) {
      float a[kRowsPerCta][4];
#pragma unroll
      for (int r = 0; r < kRowsPerCta; ++r) {
        if (b0 + r < B) load4(Ag + (int64_t)(b0 + r) * K + k, a[r]);
        else a[r][0] = a[r][1] = a[r][2] = a[r][3] = 0.f;
      }
      if (CT > 0) {
        // every class's weights are requested before the first product
        float w[CU][4];
#pragma unroll
        for (int c = 0; c < CU; ++c) load4(Wg + (int64_t)c * K + k, w[c]);
#pragma unroll
        for (int c = 0; c < CU; ++c)
#pragma unroll
          for (int r = 0; r < kRowsPerCta; ++r)
            acc[r][c] = fmaf(a[r][3], w[c][3], fmaf(a[r][2], w[c][2], fmaf(a[r][1], w[c][1], fmaf(a[r][0], w[c][0], acc[r][c]))));
      } else {
#pragma unroll
        for (int c = 0; c < CU; ++c) {
          if (c >= C) break;          // uniform: the remaining classes are skipped, not predicated off
          float w[4];
          load4(Wg + (int64_t)c * K + k, w);
#pragma unroll
          for (int r = 0; r < kRowsPerCta; ++r)
            acc[r][c] = fmaf(a[r][3], w[3], fmaf(a[r][2], w[2], fmaf(a[r][1], w[1], fmaf(a[r][0], w[0], acc[r][c]))));
        }
      }
    }
  } else {
    for (int k = kw0 + lane; k < kw1; k += 32) {
      float a[kRowsPerCta];
#pragma unroll
      for (int r = 0; r < kRowsPerCta; ++r) a[r] = (b0 + r < B) ? to_f(Ag[(int64_t)(b0 + r) * K + k]) : 0.f;
#pragma unroll
      for (int c = 0; c < CU; ++c)
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
    for (int c = 0; c < CU; ++c)
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
      s += bz;
    }
    zs[r][c] = s;
  }
  __syncthreads();
  const float invB = 1.0f / (float)B;
  if (warp < kRowsPerCta && b0 + warp < B) {
    // warp r finishes row r: lane c holds class c
    const int b = b0 + warp;
    const float z = (lane < C) ? zs[warp][lane] : -INFINITY;
    float loss, d;
    if (kind == LS_LOSS_SOFTMAX_CE) {
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
      const float res = zs[warp][0] - target;
      loss = 0.5f * res * res;
      d = res * invB;
    }
    if (lane == 0) row_loss[(int64_t)g * B + b] = loss;
    if (dZ != nullptr && lane < C) dZ[((int64_t)g * B + b) * C + lane] = d;
  }
  // training steps leave the mean of the row losses to the backward kernel of this layer
  if (defer_loss) return;
  // the last CTA of this replica adds the row losses
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

// The same layer for wide inputs (K in the thousands): one CTA = 16 mini-batch rows, warp w owns rows 2w and
// 2w + 1 over all of K, so the C x K weights are read once per 16 rows instead of once per 4 and the CTAs
// of the bf16 MLP's output layer (16 per replica) fit the GPU in one wave.  The weights of the replica are
// copied to shared memory with one batch of asynchronous copies (when they fit), and a lane requests its
// elements of eight 128-element slices of both rows before the first product: the kernel costs about two
// memory round trips.  A lane takes elements [128 u + 4 lane, + 4) of slice u.
constexpr int kWideRows = 16;
constexpr int kWideBatch = 8;             // slices of K requested together
constexpr int kWideSmemMax = 100 * 1024;  // weights staged in shared memory up to this size (two CTAs per SM)

template <typename TA, int CT>
__global__ void __launch_bounds__(kThreads, 2)
head_fwd_wide_kernel(const TA* __restrict__ A, const int64_t* __restrict__ a_row_off, const float* __restrict__ W,
                     int64_t w_gstride, const float* __restrict__ bias, const void* __restrict__ y,
                     const int64_t* __restrict__ y_row_off, float* __restrict__ dZ, float* __restrict__ row_loss,
                     float* __restrict__ loss_out, unsigned int* __restrict__ counters, int B, int K, int kind,
                     int defer_loss, int stage_w) {
  extern __shared__ float wsm[];           // [CT][K] when stage_w
  __shared__ unsigned int is_last;
  __shared__ float red[kThreads];
  grid_dep_wait();
  grid_dep_launch();
  const int g = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b0 = blockIdx.x * kWideRows + 2 * warp;          // this warp's first row
  const TA* Ag = A + ((a_row_off ? a_row_off[g] : (int64_t)g * B) + b0) * K;
  const float* Wg = W + (int64_t)g * w_gstride;
  if (stage_w) {
    const uint32_t dst = static_cast<uint32_t>(__cvta_generic_to_shared(wsm));
    for (int i = threadIdx.x; i < CT * K / 4; i += kThreads)
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + i * 16), "l"(Wg + i * 4) : "memory");
    asm volatile("cp.async.commit_group;" ::: "memory");
  }
  const float bz = (bias != nullptr && lane < CT) ? bias[(int64_t)g * w_gstride + lane] : 0.f;
  int label[2] = {0, 0};
  float target[2] = {0.f, 0.f};
  {
    const int64_t y0 = y_row_off[g] + b0;
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      if (kind == LS_LOSS_SOFTMAX_CE) label[r] = static_cast<const int32_t*>(y)[y0 + r];
      else target[r] = static_cast<const float*>(y)[y0 + r];
    }
  }
  float acc[2][CT];
#pragma unroll
  for (int r = 0; r < 2; ++r)
#pragma unroll
    for (int c = 0; c < CT; ++c) acc[r][c] = 0.f;
  const int slices = K / 128;
  for (int u0 = 0; u0 < slices; u0 += kWideBatch) {
    float a[kWideBatch][2][4];
#pragma unroll
    for (int u = 0; u < kWideBatch; ++u)
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        if (u0 + u < slices) load4(Ag + (int64_t)r * K + (u0 + u) * 128 + lane * 4, a[u][r]);
        else a[u][r][0] = a[u][r][1] = a[u][r][2] = a[u][r][3] = 0.f;
      }
    if (u0 == 0 && stage_w) {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
      __syncthreads();
    }
#pragma unroll
    for (int u = 0; u < kWideBatch; ++u) {
      if (u0 + u < slices) {
        const int k = (u0 + u) * 128 + lane * 4;
#pragma unroll
        for (int c = 0; c < CT; ++c) {
          float w[4];
          load4((stage_w ? wsm : Wg) + (int64_t)c * K + k, w);
#pragma unroll
          for (int r = 0; r < 2; ++r)
            acc[r][c] = fmaf(a[u][r][3], w[3], fmaf(a[u][r][2], w[2], fmaf(a[u][r][1], w[1], fmaf(a[u][r][0], w[0], acc[r][c]))));
        }
      }
    }
  }
  // lane sums, then lane c keeps class c of both rows
  float z[2] = {0.f, 0.f};
#pragma unroll
  for (int r = 0; r < 2; ++r)
#pragma unroll
    for (int c = 0; c < CT; ++c) {
      float v = acc[r][c];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      if (lane == c) z[r] = v + bz;
    }
  const float invB = 1.0f / (float)B;
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int b = b0 + r;
    const float zz = (lane < CT) ? z[r] : -INFINITY;
    float loss, d;
    if (kind == LS_LOSS_SOFTMAX_CE) {
      float mx = zz;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      const float e = (lane < CT) ? expf(zz - mx) : 0.f;
      float sum = e;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      const bool valid = label[r] >= 0 && label[r] < CT;
      const float zy = __shfl_sync(0xffffffffu, zz, valid ? label[r] : 0);
      loss = (mx + logf(sum)) - (valid ? zy : mx);
      d = (e / sum - (lane == label[r] ? 1.f : 0.f)) * invB;
    } else {
      const float res = __shfl_sync(0xffffffffu, zz, 0) - target[r];
      loss = 0.5f * res * res;
      d = res * invB;
    }
    if (lane == 0) row_loss[(int64_t)g * B + b] = loss;
    if (dZ != nullptr && lane < CT) dZ[((int64_t)g * B + b) * CT + lane] = d;
  }
  if (defer_loss) return;
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

__device__ __forceinline__ void load_cols(const float* p, float (&r)[1]) { r[0] = *p; }
__device__ __forceinline__ void load_cols(const __nv_bfloat16* p, float (&r)[1]) { r[0] = __bfloat162float(*p); }
__device__ __forceinline__ void load_cols(const float* p, float (&r)[2]) {
  const float2 v = *reinterpret_cast<const float2*>(p);
  r[0] = v.x; r[1] = v.y;
}
__device__ __forceinline__ void load_cols(const __nv_bfloat16* p, float (&r)[2]) {
  const __nv_bfloat162 v = *reinterpret_cast<const __nv_bfloat162*>(p);
  r[0] = __low2float(v); r[1] = __high2float(v);
}
__device__ __forceinline__ void store_cols(float* p, const float (&r)[1]) { *p = r[0]; }
__device__ __forceinline__ void store_cols(__nv_bfloat16* p, const float (&r)[1]) { *p = __float2bfloat16_rn(r[0]); }
__device__ __forceinline__ void store_cols(float* p, const float (&r)[2]) {
  *reinterpret_cast<float2*>(p) = make_float2(r[0], r[1]);
}
__device__ __forceinline__ void store_cols(__nv_bfloat16* p, const float (&r)[2]) {
  *reinterpret_cast<__nv_bfloat162*>(p) = __floats2bfloat162_rn(r[0], r[1]);
}

// One CTA = 32 * VEC columns of the layer input of one replica (VEC adjacent columns per lane); the 8
// warps take interleaved rows.  VEC = 2 needs K even and 2-element alignment and is used when it still
// leaves a CTA for every SM.  Every global operand the CTA needs (its columns of W, the W / v elements
// it will update, the biases, the first rows of A) is requested before the first wait, so the kernel
// costs about one memory round trip plus the arithmetic.  The CTA of column block 0 also adds the row
// losses that head_fwd_kernel left behind (training steps) into the mini-batch mean.
// SLAB: the CTA's columns of A (all B rows) are copied to shared memory with one batch of 16-byte
// asynchronous copies at the start, so the layer input costs one memory round trip instead of one per
// 8 * kTrip rows (needs whole column blocks, 16-byte aligned rows, and room in shared memory).
template <typename TA, int VEC, int CT, bool SLAB>
__global__ void __launch_bounds__(kThreads, 2)
head_bwd_kernel(const TA* __restrict__ A, const int64_t* __restrict__ a_row_off, const float* __restrict__ dZ,
                float* __restrict__ W, float* __restrict__ V, __nv_bfloat16* __restrict__ Wb,
                float* __restrict__ bias, float* __restrict__ vbias, int64_t w_gstride, TA* __restrict__ dPrev,
                float* __restrict__ pbias, float* __restrict__ pvbias, const float* __restrict__ row_loss,
                float* __restrict__ loss_out, int B, int C, int K, float lr, float mu) {
  constexpr int COLS = 32 * VEC;
  constexpr int kTrip = 16 / VEC;                   // rows per thread per trip
  constexpr int kUpd = (CMAX * COLS) / kThreads;    // elements of the C x COLS block per thread, at most
  constexpr int CU = CT > 0 ? CT : CMAX;            // unrolled class count
  const int CP = CT > 0 ? (CT + 3) / 4 * 4 : C;     // floats per row of dz in shared memory (16-byte rows when known)
  extern __shared__ float sm[];
  float* dz = sm;                                   // [B][CP]
  float* part = sm + (size_t)B * CP;                // [8][CMAX][COLS]
  TA* slab = reinterpret_cast<TA*>(part + 8 * CMAX * COLS);   // SLAB: [B][COLS]
  grid_dep_wait();
  grid_dep_launch();
  const int g = blockIdx.y;
  const int cx = threadIdx.x & 31, ry = threadIdx.x >> 5;
  const int k = blockIdx.x * COLS + cx * VEC;       // this thread's first column
  bool in[VEC];
#pragma unroll
  for (int v = 0; v < VEC; ++v) in[v] = k + v < K;
  const TA* Ag = A + (a_row_off ? a_row_off[g] : (int64_t)g * B) * K;
  if (SLAB) {
    constexpr int kRowBytes = COLS * (int)sizeof(TA), kPieces = kRowBytes / 16;
    const char* src = reinterpret_cast<const char*>(Ag + blockIdx.x * COLS);
    const uint32_t dst = static_cast<uint32_t>(__cvta_generic_to_shared(slab));
    for (int i = threadIdx.x; i < B * kPieces; i += kThreads) {
      const int row = i / kPieces, pc = i % kPieces;
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + row * kRowBytes + pc * 16),
                   "l"(src + (int64_t)row * K * (int)sizeof(TA) + pc * 16)
                   : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  }

  // ---- requests --------------------------------------------------------------------------------
  float wreg[CU][VEC];
#pragma unroll
  for (int c = 0; c < CU; ++c)
#pragma unroll
    for (int v = 0; v < VEC; ++v)
      wreg[c][v] = (c < C && in[v]) ? W[(int64_t)g * w_gstride + (int64_t)c * K + k + v] : 0.f;
  // update phase: thread t finishes elements t, t + 256, ... of the C x COLS block, element = (class, column)
  float wu[kUpd], vu[kUpd];
#pragma unroll
  for (int i = 0; i < kUpd; ++i) {
    const int t = threadIdx.x + i * kThreads;
    const int kk = blockIdx.x * COLS + (t % COLS);
    wu[i] = vu[i] = 0.f;
    if (t < C * COLS && kk < K) {
      const int64_t at = (int64_t)g * w_gstride + (int64_t)(t / COLS) * K + kk;
      wu[i] = W[at];
      if (mu != 0.f) vu[i] = V[at];
    }
  }
  float b_own = 0.f, vb_own = 0.f, b_prev = 0.f, vb_prev = 0.f;
  const bool own_bias = blockIdx.x == 0 && bias != nullptr && threadIdx.x < C;
  const int kp = blockIdx.x * COLS + threadIdx.x;
  const bool prev_bias = pbias != nullptr && threadIdx.x < COLS && kp < K;
  if (own_bias) {
    b_own = bias[(int64_t)g * w_gstride + threadIdx.x];
    if (mu != 0.f) vb_own = vbias[(int64_t)g * w_gstride + threadIdx.x];
  }
  if (prev_bias) {
    b_prev = pbias[(int64_t)g * w_gstride + kp];
    if (mu != 0.f) vb_prev = pvbias[(int64_t)g * w_gstride + kp];
  }
  float av[kTrip][VEC];
#pragma unroll
  for (int u = 0; u < kTrip; ++u) {
    const int b = ry + 8 * u;
#pragma unroll
    for (int v = 0; v < VEC; ++v) av[u][v] = 0.f;
    if (!SLAB && b < B && in[0]) {
      if (VEC == 1 || in[VEC - 1]) load_cols(Ag + (int64_t)b * K + k, av[u]);
      else av[u][0] = to_f(Ag[(int64_t)b * K + k]);
    }
  }
  if (blockIdx.x == 0 && ry == 7 && loss_out != nullptr) {
    // mean of the row losses: lane-strided partial sums, then a butterfly
    float p = 0.f;
    for (int b = cx; b < B; b += 32) p += row_loss[(int64_t)g * B + b];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) p += __shfl_xor_sync(0xffffffffu, p, o);
    if (cx == 0) loss_out[g] = p * (1.0f / (float)B);
  }
  for (int i = threadIdx.x; i < B * C; i += kThreads) dz[(i / C) * CP + i % C] = dZ[(int64_t)g * B * C + i];
  if (SLAB) asm volatile("cp.async.wait_group 0;" ::: "memory");
  __syncthreads();

  // ---- both gradients in one pass over the rows ------------------------------------------------------
  float gw[CU][VEC];
#pragma unroll
  for (int c = 0; c < CU; ++c)
#pragma unroll
    for (int v = 0; v < VEC; ++v) gw[c][v] = 0.f;
  float cs[VEC];      // column sums of dPrev over this thread's rows (bias gradient of the layer below)
#pragma unroll
  for (int v = 0; v < VEC; ++v) cs[v] = 0.f;
  for (int bb = 0; bb < B; bb += 8 * kTrip) {
    if (SLAB) {
#pragma unroll
      for (int u = 0; u < kTrip; ++u) {
        const int b = bb + ry + 8 * u;
#pragma unroll
        for (int v = 0; v < VEC; ++v) av[u][v] = 0.f;
        if (b < B) load_cols(slab + b * COLS + cx * VEC, av[u]);
      }
    } else if (bb > 0) {
#pragma unroll
      for (int u = 0; u < kTrip; ++u) {
        const int b = bb + ry + 8 * u;
#pragma unroll
        for (int v = 0; v < VEC; ++v) av[u][v] = 0.f;
        if (b < B && in[0]) {
          if (VEC == 1 || in[VEC - 1]) load_cols(Ag + (int64_t)b * K + k, av[u]);
          else av[u][0] = to_f(Ag[(int64_t)b * K + k]);
        }
      }
    }
#pragma unroll
    for (int u = 0; u < kTrip; ++u) {
      const int b = bb + ry + 8 * u;
      if (b >= B) break;
      float da[VEC];
#pragma unroll
      for (int v = 0; v < VEC; ++v) da[v] = 0.f;
      if (CT > 0) {
        // the row of dZ in whole 16-byte pieces, then the products: no branch between the loads
        float drow[(CU + 3) / 4 * 4];
#pragma unroll
        for (int i = 0; i < (CU + 3) / 4; ++i) {
          const float4 d4 = *reinterpret_cast<const float4*>(dz + b * CP + 4 * i);
          drow[4 * i] = d4.x; drow[4 * i + 1] = d4.y; drow[4 * i + 2] = d4.z; drow[4 * i + 3] = d4.w;
        }
#pragma unroll
        for (int c = 0; c < CU; ++c)
#pragma unroll
          for (int v = 0; v < VEC; ++v) {
            gw[c][v] = fmaf(drow[c], av[u][v], gw[c][v]);
            da[v] = fmaf(drow[c], wreg[c][v], da[v]);
          }
      } else {
#pragma unroll
        for (int c = 0; c < CU; ++c) {
          if (c >= C) break;          // uniform: the remaining classes are skipped, not predicated off
          const float d = dz[b * CP + c];
#pragma unroll
          for (int v = 0; v < VEC; ++v) {
            gw[c][v] = fmaf(d, av[u][v], gw[c][v]);
            da[v] = fmaf(d, wreg[c][v], da[v]);
          }
        }
      }
      if (dPrev != nullptr && in[0]) {
        float o[VEC];
#pragma unroll
        for (int v = 0; v < VEC; ++v) {
          o[v] = av[u][v] > 0.f ? da[v] : 0.f;
          cs[v] += o[v];
        }
        TA* dst = dPrev + ((int64_t)g * B + b) * K + k;
        if (VEC == 1 || in[VEC - 1]) store_cols(dst, o);
        else put(dst, o[0]);
      }
    }
  }
#pragma unroll
  for (int c = 0; c < CU; ++c)
#pragma unroll
    for (int v = 0; v < VEC; ++v) part[(ry * CMAX + c) * COLS + cx * VEC + v] = gw[c][v];
  __syncthreads();
  // ---- G = sum of the 8 row slices (in slice order); v <- mu v + G; W <- W - eta v -------------------
#pragma unroll
  for (int i = 0; i < kUpd; ++i) {
    const int t = threadIdx.x + i * kThreads;
    const int c = t / COLS, col = t % COLS;
    const int kk = blockIdx.x * COLS + col;
    if (t < C * COLS && kk < K) {
      float s = 0.f;
#pragma unroll
      for (int r = 0; r < 8; ++r) s += part[(r * CMAX + c) * COLS + col];
      const int64_t at = (int64_t)g * w_gstride + (int64_t)c * K + kk;
      float step = s;
      if (mu != 0.f) {
        step = fmaf(mu, vu[i], s);
        V[at] = step;
      }
      const float w = fmaf(-lr, step, wu[i]);
      W[at] = w;
      if (Wb != nullptr) Wb[at] = __float2bfloat16_rn(w);
    }
  }
  if (own_bias) {
    const int c = threadIdx.x;
    float s = 0.f;
    for (int b = 0; b < B; ++b) s += dz[b * CP + c];
    const int64_t at = (int64_t)g * w_gstride + c;
    float step = s;
    if (mu != 0.f) {
      step = fmaf(mu, vb_own, s);
      vbias[at] = step;
    }
    bias[at] = fmaf(-lr, step, b_own);
  }
  if (pbias != nullptr) {
    // bias of the layer below: its gradient is the column sum of dPrev, complete inside this CTA
    __syncthreads();
#pragma unroll
    for (int v = 0; v < VEC; ++v) part[ry * COLS + cx * VEC + v] = cs[v];
    __syncthreads();
    if (prev_bias) {
      float s = 0.f;
#pragma unroll
      for (int r = 0; r < 8; ++r) s += part[r * COLS + threadIdx.x];
      const int64_t at = (int64_t)g * w_gstride + kp;
      float step = s;
      if (mu != 0.f) {
        step = fmaf(mu, vb_prev, s);
        pvbias[at] = step;
      }
      pbias[at] = fmaf(-lr, step, b_prev);
    }
  }
}

}  // namespace

bool head_shape_ok(int B, int C) { return C >= 1 && C <= CMAX && B >= 1 && (size_t)B * C * 4 <= 64 * 1024; }

template <typename TA, int CT>
int launch_head_fwd_wide(const HeadFwdArgs& a, cudaStream_t st) {
  auto kern = head_fwd_wide_kernel<TA, CT>;
  static uint64_t configured = 0;        // one bit per device
  {
    cudaError_t e = allow_dynamic_smem(kern, (int)(kWideSmemMax), &configured);
    if (e != cudaSuccess) return e;
  }
  const size_t wbytes = (size_t)CT * a.K * sizeof(float);
  const int stage_w = wbytes <= (size_t)kWideSmemMax ? 1 : 0;
  dim3 grid((unsigned)(a.B / kWideRows), (unsigned)a.groups);
  return launch_dep(kern, grid, dim3(kThreads), stage_w ? wbytes : 0, st, 1, static_cast<const TA*>(a.A),
                    a.a_row_off, a.W, a.w_gstride, a.bias, a.y, a.y_row_off, a.dZ, a.row_loss, a.loss_out, a.counters,
                    a.B, a.K, a.loss_kind, a.defer_loss, stage_w);
}

int launch_head_fwd(const HeadFwdArgs& a, bool a_bf16, cudaStream_t st, int64_t* launches) {
  if (launches) ++*launches;
  // wide inputs with enough rows to fill the GPU 16 at a time: the kernel that reads W once per 16 rows
  if ((a.C == 10 || a.C == 1) && a.K >= 1024 && a.K % 128 == 0 && a.B % kWideRows == 0 &&
      (int64_t)(a.B / kWideRows) * a.groups >= 64 && reinterpret_cast<uintptr_t>(a.A) % 16 == 0 &&
      reinterpret_cast<uintptr_t>(a.W) % 16 == 0 && a.w_gstride % 4 == 0) {
    if (a_bf16) return a.C == 10 ? launch_head_fwd_wide<__nv_bfloat16, 10>(a, st) : launch_head_fwd_wide<__nv_bfloat16, 1>(a, st);
    return a.C == 10 ? launch_head_fwd_wide<float, 10>(a, st) : launch_head_fwd_wide<float, 1>(a, st);
  }
  dim3 grid((unsigned)((a.B + kRowsPerCta - 1) / kRowsPerCta), (unsigned)a.groups);
  const int vec_ok = (a.K % 4 == 0) && (reinterpret_cast<uintptr_t>(a.A) % 16 == 0) &&
                     (reinterpret_cast<uintptr_t>(a.W) % 16 == 0) && (a.w_gstride % 4 == 0);
  if (a_bf16) {
    auto go = [&](auto kern) {
      return launch_dep(kern, grid, dim3(kThreads), 0, st, 1, static_cast<const __nv_bfloat16*>(a.A), a.a_row_off, a.W,
                        a.w_gstride, a.bias, a.y, a.y_row_off, a.dZ, a.row_loss, a.loss_out, a.counters, a.B, a.C, a.K,
                        a.loss_kind, vec_ok, a.defer_loss);
    };
    if (a.C == 10) return go(head_fwd_kernel<__nv_bfloat16, 10>);
    if (a.C == 1) return go(head_fwd_kernel<__nv_bfloat16, 1>);
    return go(head_fwd_kernel<__nv_bfloat16, 0>);
  }
  auto go = [&](auto kern) {
    return launch_dep(kern, grid, dim3(kThreads), 0, st, 1, static_cast<const float*>(a.A), a.a_row_off, a.W,
                      a.w_gstride, a.bias, a.y, a.y_row_off, a.dZ, a.row_loss, a.loss_out, a.counters, a.B, a.C, a.K,
                      a.loss_kind, vec_ok, a.defer_loss);
  };
  if (a.C == 10) return go(head_fwd_kernel<float, 10>);
  if (a.C == 1) return go(head_fwd_kernel<float, 1>);
  return go(head_fwd_kernel<float, 0>);
}

template <typename TA, int VEC, int CT, bool SLAB>
int launch_head_bwd_s(const HeadBwdArgs& a, size_t smem, cudaStream_t st) {
  auto kern = head_bwd_kernel<TA, VEC, CT, SLAB>;
  static uint64_t configured = 0;        // one bit per device
  {
    cudaError_t e = allow_dynamic_smem(kern, (int)(112 * 1024), &configured);
    if (e != cudaSuccess) return e;
  }
  constexpr int COLS = 32 * VEC;
  dim3 grid((unsigned)((a.K + COLS - 1) / COLS), (unsigned)a.groups);
  return launch_dep(kern, grid, dim3(kThreads), smem, st, 1, static_cast<const TA*>(a.A), a.a_row_off, a.dZ, a.W, a.V,
                    a.Wb, a.bias, a.vbias, a.w_gstride, static_cast<TA*>(a.dPrev), a.dPrev ? a.pbias : nullptr,
                    a.pvbias, a.row_loss, a.loss_out, a.B, a.C, a.K, a.lr, a.mu);
}

template <typename TA, int VEC, int CT>
int launch_head_bwd_c(const HeadBwdArgs& a, cudaStream_t st) {
  constexpr int COLS = 32 * VEC;
  const size_t base = ((size_t)a.B * (CT > 0 ? (CT + 3) / 4 * 4 : a.C) + 8 * CMAX * COLS) * sizeof(float);
  const size_t slab = (size_t)a.B * COLS * sizeof(TA);
  // the slab variant: whole column blocks, rows that start on 16-byte boundaries, two CTAs per SM still fit
  const bool ok = COLS * sizeof(TA) % 16 == 0 && a.K % COLS == 0 && ((size_t)a.K * sizeof(TA)) % 16 == 0 &&
                  reinterpret_cast<uintptr_t>(a.A) % 16 == 0 && base % 16 == 0 && base + slab <= 100 * 1024;
  if (ok) return launch_head_bwd_s<TA, VEC, CT, true>(a, base + slab, st);
  return launch_head_bwd_s<TA, VEC, CT, false>(a, base, st);
}

template <typename TA, int VEC>
int launch_head_bwd_t(const HeadBwdArgs& a, cudaStream_t st) {
  if (a.C == 10) return launch_head_bwd_c<TA, VEC, 10>(a, st);
  if (a.C == 1) return launch_head_bwd_c<TA, VEC, 1>(a, st);
  return launch_head_bwd_c<TA, VEC, 0>(a, st);
}

int launch_head_bwd(const HeadBwdArgs& a, bool a_bf16, cudaStream_t st, int64_t* launches) {
  if (launches) ++*launches;
  const size_t esz = a_bf16 ? 2 : 4;
  // two columns per lane when the pointers allow it and there is still a CTA for every SM
  const bool pair = (a.K % 2 == 0) && reinterpret_cast<uintptr_t>(a.A) % (2 * esz) == 0 &&
                    (a.dPrev == nullptr || reinterpret_cast<uintptr_t>(a.dPrev) % (2 * esz) == 0) &&
                    (int64_t)((a.K + 63) / 64) * a.groups >= 148;
  if (a_bf16) return pair ? launch_head_bwd_t<__nv_bfloat16, 2>(a, st) : launch_head_bwd_t<__nv_bfloat16, 1>(a, st);
  return pair ? launch_head_bwd_t<float, 2>(a, st) : launch_head_bwd_t<float, 1>(a, st);
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

// What must be fresh at every call: the CTA counters start at zero and chunk c starts at row c * chunk_rows.
// (Device code names the array directly.)  A kernel rather than host-to-device copies: the call enqueues
// nothing that reads host memory later.
__global__ void static_scratch_reset_kernel(int chunks, int chunk_rows) {
  StaticScratch* sc = reinterpret_cast<StaticScratch*>(g_static_scratch);
  for (int c = threadIdx.x; c < kStaticMaxChunks; c += blockDim.x) {
    sc->counters[c] = 0u;
    if (c < chunks) sc->row_off[c] = (long long)c * chunk_rows;
  }
}

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
  static_scratch_reset_kernel<<<1, 256, 0, st>>>((int)chunks, chunk_rows);
  if (cudaGetLastError() != cudaSuccess) return LS_ERR_CUDA;
  HeadFwdArgs a;
  a.A = x_dev; a.a_row_off = reinterpret_cast<const int64_t*>(sc->row_off);
  a.W = W_dev; a.w_gstride = 0; a.bias = bias_dev;
  a.y = y_dev; a.y_row_off = reinterpret_cast<const int64_t*>(sc->row_off);
  a.dZ = nullptr;
  a.row_loss = sc->row_loss; a.loss_out = chunk_loss_dev; a.counters = sc->counters;
  a.B = chunk_rows; a.C = d_out; a.K = d_in; a.groups = (int)chunks; a.loss_kind = loss;
  a.defer_loss = 0;
  return launch_head_fwd(a, false, st, nullptr) == cudaSuccess ? LS_OK : LS_ERR_CUDA;
}
