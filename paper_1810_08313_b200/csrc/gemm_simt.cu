// Grouped (one group per replica) matrix products on the fp32 CUDA cores with
// the layer arithmetic fused into the epilogues.  These kernels carry every
// shape: the fp32 models, and in bf16 models the layers whose width does not
// fill a tensor-core tile (the 10-wide loss layer).  Accumulation is fp32 in a
// fixed k order, so results are reproducible run to run.
//
//   forward   Z = A W^T + b, A_l = relu(Z)                (evaluating f, Section 2)
//   backward  dZ_{l-1} = (dZ_l W_l) * 1[A_{l-1} > 0]
//   update    G = dZ^T A ; v <- mu v + G ; W <- W - eta v  (Section 2 mini-batch SGD
//             update; Section 5.3 momentum)  -- G is never written to memory.
#include "ls_internal.h"

namespace ls {
namespace {

constexpr int BM = 64, BN = 64, BK = 16, PAD = 4;
constexpr int kThreads = 256;

__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(__nv_bfloat16 v) { return __bfloat162float(v); }

__device__ __forceinline__ void load_vec4(const float* p, float (&r)[4]) {
  float4 v = *reinterpret_cast<const float4*>(p);
  r[0] = v.x; r[1] = v.y; r[2] = v.z; r[3] = v.w;
}
__device__ __forceinline__ void load_vec4(const __nv_bfloat16* p, float (&r)[4]) {
  uint2 u = *reinterpret_cast<const uint2*>(p);
  __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162*>(&u.x);
  __nv_bfloat162 b = *reinterpret_cast<__nv_bfloat162*>(&u.y);
  r[0] = __low2float(a); r[1] = __high2float(a); r[2] = __low2float(b); r[3] = __high2float(b);
}
__device__ __forceinline__ void store_out(float* p, float v) { *p = v; }
__device__ __forceinline__ void store_out(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }
__device__ __forceinline__ void store_out4(float* p, const float (&v)[4]) {
  *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
}
__device__ __forceinline__ void store_out4(__nv_bfloat16* p, const float (&v)[4]) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(v[0], v[1]);
  __nv_bfloat162 hi = __floats2bfloat162_rn(v[2], v[3]);
  uint2 u;
  u.x = *reinterpret_cast<uint32_t*>(&lo);
  u.y = *reinterpret_cast<uint32_t*>(&hi);
  *reinterpret_cast<uint2*>(p) = u;
}

// One operand of the product, seen as a (rows x K) matrix: element (r, k) is
// at base + r*ld + k when K_CONTIG, at base + k*ld + r otherwise.
template <typename T, bool K_CONTIG>
struct Operand {
  const T* base;
  int64_t ld;
  int rows, K;
  bool vec;   // 4-element vector loads are legal (alignment checked on the host)

  __device__ __forceinline__ void fetch(int r0, int k0, int tid, float (&reg)[4]) const {
    if (K_CONTIG) {
      const int r = r0 + (tid >> 2), k = k0 + (tid & 3) * 4;
      if (r < rows && vec && k + 3 < K) {
        load_vec4(base + (int64_t)r * ld + k, reg);
      } else {
#pragma unroll
        for (int s = 0; s < 4; ++s) reg[s] = (r < rows && k + s < K) ? to_f(base[(int64_t)r * ld + k + s]) : 0.f;
      }
    } else {
      const int k = k0 + (tid >> 4), r = r0 + (tid & 15) * 4;
      if (k < K && vec && r + 3 < rows) {
        load_vec4(base + (int64_t)k * ld + r, reg);
      } else {
#pragma unroll
        for (int s = 0; s < 4; ++s) reg[s] = (k < K && r + s < rows) ? to_f(base[(int64_t)k * ld + r + s]) : 0.f;
      }
    }
  }
  // shared tile is [BK][rows_in_tile + PAD]
  __device__ __forceinline__ void stash(float (*sm)[BM + PAD], int tid, const float (&reg)[4]) const {
    if (K_CONTIG) {
      const int r = tid >> 2, k = (tid & 3) * 4;
#pragma unroll
      for (int s = 0; s < 4; ++s) sm[k + s][r] = reg[s];
    } else {
      const int k = tid >> 4, r = (tid & 15) * 4;
      *reinterpret_cast<float4*>(&sm[k][r]) = make_float4(reg[0], reg[1], reg[2], reg[3]);
    }
  }
};

template <typename TA, bool A_KC, typename TB, bool B_KC, class Epi>
__global__ void __launch_bounds__(kThreads)
gemm_kernel(const TA* A, int64_t a_gstride, const int64_t* a_row_off, int64_t lda, bool a_vec,
            const TB* B, int64_t b_gstride, const int64_t* b_row_off, int64_t ldb, bool b_vec,
            int M, int N, int K, Epi epi) {
  static_assert(BM == BN, "square tiles");
  __shared__ __align__(16) float As[BK][BM + PAD];
  __shared__ __align__(16) float Bs[BK][BN + PAD];
  grid_dep_wait();
  grid_dep_launch();
  const int g = blockIdx.z;
  const int i0 = blockIdx.y * BM, j0 = blockIdx.x * BN;
  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;

  Operand<TA, A_KC> opA{A + (a_row_off ? a_row_off[g] * lda : (int64_t)g * a_gstride), lda, M, K, a_vec};
  Operand<TB, B_KC> opB{B + (b_row_off ? b_row_off[g] * ldb : (int64_t)g * b_gstride), ldb, N, K, b_vec};

  float acc[4][4];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;

  float ra[4], rb[4];
  opA.fetch(i0, 0, tid, ra);
  opB.fetch(j0, 0, tid, rb);
  for (int k0 = 0; k0 < K; k0 += BK) {
    opA.stash(As, tid, ra);
    opB.stash(Bs, tid, rb);
    __syncthreads();
    if (k0 + BK < K) {
      opA.fetch(i0, k0 + BK, tid, ra);
      opB.fetch(j0, k0 + BK, tid, rb);
    }
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      const float4 a = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
      const float4 b = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
      const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int x = 0; x < 4; ++x)
#pragma unroll
        for (int y = 0; y < 4; ++y) acc[x][y] = fmaf(av[x], bv[y], acc[x][y]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int x = 0; x < 4; ++x) {
    const int i = i0 + ty * 4 + x;
    const int j = j0 + tx * 4;
    if (i < M && j < N) epi(g, i, j, acc[x], min(4, N - j));
  }
}

// ---- epilogues ---------------------------------------------------------------

template <typename TC>
struct EpiFwd {
  const float* bias; int64_t bias_gstride;
  TC* C; int M, N; int relu; bool vec;
  __device__ __forceinline__ void operator()(int g, int i, int j, const float (&acc)[4], int nv) const {
    float o[4];
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      float v = acc[s];
      if (bias != nullptr && s < nv) v += bias[(int64_t)g * bias_gstride + j + s];
      o[s] = (relu && !(v > 0.f)) ? 0.f : v;
    }
    const int64_t at = ((int64_t)g * M + i) * N + j;
    TC* p = C + at;
    if (vec && nv == 4) store_out4(p, o);
    else for (int s = 0; s < nv; ++s) store_out(p + s, o[s]);
  }
};

template <typename TC>
struct EpiDx {
  const TC* act; TC* C; int M, N; bool vec;
  __device__ __forceinline__ void operator()(int g, int i, int j, const float (&acc)[4], int nv) const {
    const int64_t at = ((int64_t)g * M + i) * N + j;
    float o[4];
#pragma unroll
    for (int s = 0; s < 4; ++s) o[s] = (s < nv && to_f(act[at + s]) > 0.f) ? acc[s] : 0.f;
    if (vec && nv == 4) store_out4(C + at, o);
    else for (int s = 0; s < nv; ++s) store_out(C + at + s, o[s]);
  }
};

struct EpiDw {
  float* W; float* V; __nv_bfloat16* Wb; int64_t gstride; int N; float lr, mu; bool vec;
  __device__ __forceinline__ void operator()(int g, int i, int j, const float (&acc)[4], int nv) const {
    const int64_t at = (int64_t)g * gstride + (int64_t)i * N + j;
    float w[4], v[4];
    if (vec && nv == 4) {
      load_vec4(W + at, w);
      if (mu != 0.f) load_vec4(V + at, v);
    } else {
      for (int s = 0; s < nv; ++s) { w[s] = W[at + s]; if (mu != 0.f) v[s] = V[at + s]; }
    }
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      const float step = (mu != 0.f) ? fmaf(mu, v[s], acc[s]) : acc[s];
      v[s] = step;
      w[s] = fmaf(-lr, step, w[s]);
    }
    if (vec && nv == 4) {
      store_out4(W + at, w);
      if (mu != 0.f) store_out4(V + at, v);
      if (Wb != nullptr) store_out4(Wb + at, w);
    } else {
      for (int s = 0; s < nv; ++s) {
        W[at + s] = w[s];
        if (mu != 0.f) V[at + s] = v[s];
        if (Wb != nullptr) Wb[at + s] = __float2bfloat16_rn(w[s]);
      }
    }
  }
};

inline bool aligned(const void* p, size_t a) { return reinterpret_cast<uintptr_t>(p) % a == 0; }

template <typename T>
inline bool can_vec(const void* base, int64_t ld, int64_t gstride) {
  // 4-element vectors: 16 bytes for float, 8 for bf16
  return aligned(base, 4 * sizeof(T)) && ld % 4 == 0 && gstride % 4 == 0;
}

inline dim3 grid_for(int M, int N, int groups) {
  return dim3((unsigned)((N + BN - 1) / BN), (unsigned)((M + BM - 1) / BM), (unsigned)groups);
}

template <typename TA, typename TW, typename TC>
int fwd_typed(const FwdArgs& a, cudaStream_t st) {
  const TA* A = static_cast<const TA*>(a.A);
  const TW* W = static_cast<const TW*>(a.W);
  EpiFwd<TC> epi{a.bias, a.bias_gstride, static_cast<TC*>(a.C), a.M, a.N, a.relu,
                 aligned(a.C, 4 * sizeof(TC)) && a.N % 4 == 0};
  const int64_t a_gs = (int64_t)a.M * a.K;
  return launch_dep(gemm_kernel<TA, true, TW, true, EpiFwd<TC>>, grid_for(a.M, a.N, a.groups), dim3(kThreads), 0, st, 1,
                    A, a_gs, a.row_off, a.K, can_vec<TA>(A, a.K, a_gs), W, a.w_gstride, nullptr, a.K,
                    can_vec<TW>(W, a.K, a.w_gstride), a.M, a.N, a.K, epi);
}

template <typename T>
int dx_typed(const DxArgs& a, cudaStream_t st) {
  const T* dZ = static_cast<const T*>(a.dZ);
  const T* W = static_cast<const T*>(a.W);
  EpiDx<T> epi{static_cast<const T*>(a.act), static_cast<T*>(a.C), a.M, a.N,
               aligned(a.C, 4 * sizeof(T)) && aligned(a.act, 4 * sizeof(T)) && a.N % 4 == 0};
  const int64_t a_gs = (int64_t)a.M * a.K;
  return launch_dep(gemm_kernel<T, true, T, false, EpiDx<T>>, grid_for(a.M, a.N, a.groups), dim3(kThreads), 0, st, 1,
                    dZ, a_gs, nullptr, a.K, can_vec<T>(dZ, a.K, a_gs), W, a.w_gstride, nullptr, a.N,
                    can_vec<T>(W, a.N, a.w_gstride), a.M, a.N, a.K, epi);
}

template <typename T>
int dw_typed(const DwArgs& a, cudaStream_t st) {
  const T* dZ = static_cast<const T*>(a.dZ);
  const T* A = static_cast<const T*>(a.A);
  EpiDw epi{a.W, a.V, a.Wb, a.w_gstride, a.N, a.lr, a.mu,
            aligned(a.W, 16) && aligned(a.V, 16) && (a.Wb == nullptr || aligned(a.Wb, 8)) && a.N % 4 == 0 &&
                a.w_gstride % 4 == 0};
  const int64_t dz_gs = (int64_t)a.B * a.M, a_gs = (int64_t)a.B * a.N;
  return launch_dep(gemm_kernel<T, false, T, false, EpiDw>, grid_for(a.M, a.N, a.groups), dim3(kThreads), 0, st, 1,
                    dZ, dz_gs, nullptr, a.M, can_vec<T>(dZ, a.M, dz_gs), A, a_gs, a.row_off, a.N,
                    can_vec<T>(A, a.N, a_gs), a.M, a.N, a.B, epi);
}

}  // namespace

int launch_fwd(const FwdArgs& a, bool a_bf16, bool w_bf16, bool c_bf16, cudaStream_t st, int64_t* launches) {
  if (launches) ++*launches;
  if (!a_bf16 && !w_bf16 && !c_bf16) return fwd_typed<float, float, float>(a, st);
  if (a_bf16 && w_bf16 && c_bf16) return fwd_typed<__nv_bfloat16, __nv_bfloat16, __nv_bfloat16>(a, st);
  if (a_bf16 && w_bf16 && !c_bf16) return fwd_typed<__nv_bfloat16, __nv_bfloat16, float>(a, st);
  return cudaErrorInvalidValue;
}
int launch_dx(const DxArgs& a, bool bf16, cudaStream_t st, int64_t* launches) {
  if (launches) ++*launches;
  return bf16 ? dx_typed<__nv_bfloat16>(a, st) : dx_typed<float>(a, st);
}
int launch_dw(const DwArgs& a, bool bf16, cudaStream_t st, int64_t* launches) {
  if (launches) ++*launches;
  return bf16 ? dw_typed<__nv_bfloat16>(a, st) : dw_typed<float>(a, st);
}

}  // namespace ls
