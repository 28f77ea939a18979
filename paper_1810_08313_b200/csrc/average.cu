// Model averaging: X <- X J, J = 1 1^T / m (Section 2, PASGD update rule, the
// case k mod tau = 0; operator J of the convergence proof's notation).
//
// Bandwidth-bound streaming kernel.  Every thread owns one 32-byte column slice
// (eight floats; sixteen bytes when the buffers are only 16-byte aligned): it
// issues the m independent 256-bit loads of that slice, one per replica, before
// using any of them, adds them in replica order in fp32, divides once by
// (float)m and stores the mean back to all m replicas.  One slice per thread
// and a grid that covers the vector exactly: measured on B200 this streams
// faster than a persistent grid-stride loop (the hardware scheduler keeps more
// independent loads in flight than a loop that reuses its registers).
// Algorithmic traffic is 8*m bytes per parameter: each element is read once and
// written once.  No shared memory, no inter-thread communication: the reduction
// order is fixed by construction, so the result is bit-reproducible.
//
// Block momentum (Section 5.3) is the same pass with two more streams: the model
// the period started from (anchor) and the global buffer u.  With mean the average
// above, d = anchor - mean, G = d / eta, u' = beta*u + G, x' = anchor - eta*u', every
// operation rounded separately; x' goes to all replicas and the anchor, u' to u.
// Traffic grows from 8m to 8m + 16 bytes per parameter.
#include "ls_internal.h"

namespace ls {

namespace {

constexpr int kThreads = 256;
constexpr int kMaxPieces = LS_MAX_LAYERS + 1;

template <int W> struct Vec;
template <> struct Vec<4> {
  float v[4];
  __device__ __forceinline__ void load(const float* p) {
    const float4 t = __ldcs(reinterpret_cast<const float4*>(p));
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
  }
  __device__ __forceinline__ void store(float* p) const {
    *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
  }
};
template <> struct Vec<8> {
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

template <int W>
__device__ __forceinline__ void store_bf16(__nv_bfloat16* p, const float (&v)[W]) {
  uint32_t u[W / 2];
#pragma unroll
  for (int e = 0; e < W / 2; ++e) {
    __nv_bfloat162 t = __floats2bfloat162_rn(v[2 * e], v[2 * e + 1]);
    u[e] = *reinterpret_cast<uint32_t*>(&t);
  }
  if constexpr (W == 8) *reinterpret_cast<uint4*>(p) = make_uint4(u[0], u[1], u[2], u[3]);
  else *reinterpret_cast<uint2*>(p) = make_uint2(u[0], u[1]);
}

// M > 0: replica count known at compile time (all m loads in flight at once).
// M == 0: any m, processed in chunks of 8 replicas, still in replica order.
// W: floats per thread (8 or 4).  Plain IEEE adds and one IEEE division: there is no
// multiply nearby, so nothing can be contracted into an FMA.
// BM: block momentum; bm.anchor / bm.u are single vectors laid out like one replica.
template <int M, int W, bool BM>
__global__ void __launch_bounds__(kThreads)
average_kernel(float* __restrict__ base, int64_t buf_stride, int m_rt, int64_t n_vec, int64_t stride,
               __nv_bfloat16* __restrict__ shadow, BlockMomentum bm, float* __restrict__ sync_out, int64_t sync_stride,
               TileMap tiles) {
  grid_dep_wait();
  grid_dep_launch();
  const int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x;
  if (i >= n_vec) return;
  const int m = M > 0 ? M : m_rt;
  float* p = base + (int64_t)blockIdx.y * buf_stride + i * W;
  const float mf = (float)m;
  Vec<W> s, anc, ug;
  if constexpr (BM) {
    anc.load(bm.anchor + i * W);
    ug.load(bm.u + i * W);
  }
  if (M > 0) {
    Vec<W> v[M > 0 ? M : 1];
#pragma unroll
    for (int j = 0; j < M; ++j) v[j].load(p + (int64_t)j * stride);
    s = v[0];
#pragma unroll
    for (int j = 1; j < M; ++j)
#pragma unroll
      for (int e = 0; e < W; ++e) s.v[e] = __fadd_rn(s.v[e], v[j].v[e]);
  } else {
    s.load(p);
    for (int j0 = 1; j0 < m; j0 += 8) {
      Vec<W> v[8];
#pragma unroll
      for (int j = 0; j < 8; ++j)
        if (j0 + j < m) v[j].load(p + (int64_t)(j0 + j) * stride);
#pragma unroll
      for (int j = 0; j < 8; ++j)
        if (j0 + j < m)
#pragma unroll
          for (int e = 0; e < W; ++e) s.v[e] = __fadd_rn(s.v[e], v[j].v[e]);
    }
  }
#pragma unroll
  for (int e = 0; e < W; ++e) s.v[e] = __fdiv_rn(s.v[e], mf);
  if constexpr (BM) {
#pragma unroll
    for (int e = 0; e < W; ++e) {
      const float d = __fsub_rn(anc.v[e], s.v[e]);
      const float G = __fdiv_rn(d, bm.lr);
      const float un = __fadd_rn(__fmul_rn(bm.beta, ug.v[e]), G);
      ug.v[e] = un;
      s.v[e] = __fsub_rn(anc.v[e], __fmul_rn(bm.lr, un));
    }
    ug.store(bm.u + i * W);
    s.store(bm.anchor + i * W);
  }
#pragma unroll 4
  for (int j = 0; j < m; ++j) s.store(p + (int64_t)j * stride);
  // the synchronized copy: what every replica holds now (read by the next local step while they are still equal)
  if (sync_out != nullptr) s.store(sync_out + (int64_t)blockIdx.y * sync_stride + i * W);
  if (blockIdx.y == 0 && shadow != nullptr) {
    const int64_t at = shadow_index(tiles, i * W);
    for (int j = 0; j < m; ++j) store_bf16<W>(shadow + (int64_t)j * stride + at, s.v);
  }
}

// Scalar path: the ragged tail (n mod W elements) and buffers that are not
// 16-byte aligned.  Same arithmetic, one element per thread.
__global__ void __launch_bounds__(kThreads)
average_scalar_kernel(float* __restrict__ base, int64_t buf_stride, int m, int64_t first, int64_t n, int64_t stride,
                      __nv_bfloat16* __restrict__ shadow, BlockMomentum bm, float* __restrict__ sync_out,
                      int64_t sync_stride, TileMap tiles) {
  grid_dep_wait();
  grid_dep_launch();
  float* buf = base + (int64_t)blockIdx.y * buf_stride;
  const float mf = (float)m;
  const int64_t i = first + (int64_t)blockIdx.x * kThreads + threadIdx.x;
  if (i >= n) return;
  float s = buf[i];
  for (int j = 1; j < m; ++j) s = __fadd_rn(s, buf[(int64_t)j * stride + i]);
  float mean = __fdiv_rn(s, mf);
  if (bm.anchor != nullptr) {
    const float a = bm.anchor[i];
    const float G = __fdiv_rn(__fsub_rn(a, mean), bm.lr);
    const float un = __fadd_rn(__fmul_rn(bm.beta, bm.u[i]), G);
    bm.u[i] = un;
    mean = __fsub_rn(a, __fmul_rn(bm.lr, un));
    bm.anchor[i] = mean;
  }
  for (int j = 0; j < m; ++j) buf[(int64_t)j * stride + i] = mean;
  if (sync_out != nullptr) sync_out[(int64_t)blockIdx.y * sync_stride + i] = mean;
  if (blockIdx.y == 0 && shadow != nullptr) {
    const int64_t at = shadow_index(tiles, i);
    for (int j = 0; j < m; ++j) shadow[(int64_t)j * stride + at] = __float2bfloat16_rn(mean);
  }
}

// The same pass over several short pieces of the replica vectors in ONE launch (the biases and narrow layers
// between the matrices that the step + averaging kernel owns): piece r covers elements [begin[r], begin[r] + 8 len[r])
// and thread i of the launch takes 8-float slice i - first[r] of the piece with first[r] <= i < first[r + 1].
// Arithmetic and order are those of average_kernel<0, 8, false>.
struct Pieces {
  int n;
  int64_t begin[kMaxPieces];
  int64_t first[kMaxPieces + 1];
};
__global__ void __launch_bounds__(kThreads)
average_pieces_kernel(float* __restrict__ base, int64_t buf_stride, int m, Pieces pc, int64_t stride,
                      __nv_bfloat16* __restrict__ shadow, float* __restrict__ sync_out, int64_t sync_stride) {
  grid_dep_wait();
  grid_dep_launch();
  const int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x;
  if (i >= pc.first[pc.n]) return;
  int r = 0;
#pragma unroll
  for (int k = 1; k < kMaxPieces; ++k)
    if (k < pc.n && i >= pc.first[k]) r = k;
  const int64_t at = pc.begin[r] + (i - pc.first[r]) * 8;
  float* p = base + (int64_t)blockIdx.y * buf_stride + at;
  const float mf = (float)m;
  Vec<8> s;
  s.load(p);
  for (int j0 = 1; j0 < m; j0 += 8) {
    Vec<8> v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j)
      if (j0 + j < m) v[j].load(p + (int64_t)(j0 + j) * stride);
#pragma unroll
    for (int j = 0; j < 8; ++j)
      if (j0 + j < m)
#pragma unroll
        for (int e = 0; e < 8; ++e) s.v[e] = __fadd_rn(s.v[e], v[j].v[e]);
  }
#pragma unroll
  for (int e = 0; e < 8; ++e) s.v[e] = __fdiv_rn(s.v[e], mf);
#pragma unroll 4
  for (int j = 0; j < m; ++j) s.store(p + (int64_t)j * stride);
  if (sync_out != nullptr) s.store(sync_out + (int64_t)blockIdx.y * sync_stride + at);
  if (blockIdx.y == 0 && shadow != nullptr)
    for (int j = 0; j < m; ++j) store_bf16<8>(shadow + (int64_t)j * stride + at, s.v);
}

template <int W, bool BM>
void launch_vec(dim3 grid, cudaStream_t st, float* base, int64_t buf_stride, int m, int64_t n_vec, int64_t stride,
                __nv_bfloat16* shadow, const BlockMomentum& bm, float* sync_out, int64_t sync_stride, const TileMap& tiles) {
#define LS_AVG(M) launch_dep(average_kernel<M, W, BM>, grid, dim3(kThreads), 0, st, 1, base, buf_stride, m, n_vec, stride, shadow, bm, sync_out, sync_stride, tiles)
  switch (m) {
    case 2: LS_AVG(2); break;
    case 4: LS_AVG(4); break;
    case 8: LS_AVG(8); break;
    case 16: LS_AVG(16); break;
    default: LS_AVG(0); break;
  }
#undef LS_AVG
}

inline bool aligned_to(const void* p, size_t a) { return p == nullptr || reinterpret_cast<uintptr_t>(p) % a == 0; }

}  // namespace

int launch_average(float* base, int n_buf, int64_t buf_stride, int m, int64_t n, int64_t stride,
                   __nv_bfloat16* shadow, cudaStream_t st, int64_t* launches, const BlockMomentum* bmp, float* sync_out,
                   int64_t sync_stride, const TileMap* tilesp) {
  if (sync_stride <= 0) sync_stride = n;
  const TileMap tiles = tilesp ? *tilesp : TileMap{};
  if (n <= 0 || n_buf <= 0) return cudaSuccess;
  BlockMomentum bm{nullptr, nullptr, 0.f, 0.f};
  if (bmp != nullptr) {
    if (n_buf != 1 || bmp->anchor == nullptr || bmp->u == nullptr) return cudaErrorInvalidValue;
    bm = *bmp;
  }
  const bool BM = bm.anchor != nullptr;
  // widest slice the addresses allow: 8 floats (32-byte aligned), 4 floats (16-byte), else scalar
  int W = 0;
  if (aligned_to(base, 32) && stride % 8 == 0 && buf_stride % 8 == 0 && aligned_to(shadow, 16) &&
      aligned_to(bm.anchor, 32) && aligned_to(bm.u, 32) && aligned_to(sync_out, 32))
    W = 8;
  else if (aligned_to(base, 16) && stride % 4 == 0 && buf_stride % 4 == 0 && aligned_to(shadow, 8) &&
           aligned_to(bm.anchor, 16) && aligned_to(bm.u, 16) && aligned_to(sync_out, 16))
    W = 4;
  const int64_t n_vec = W ? n / W : 0;
  if (n_vec > 0) {
    const int64_t gx = (n_vec + kThreads - 1) / kThreads;
    if (gx > 2147483647LL) return cudaErrorInvalidValue;
    dim3 grid((unsigned)gx, (unsigned)n_buf);
    if (W == 8) {
      if (BM) launch_vec<8, true>(grid, st, base, buf_stride, m, n_vec, stride, shadow, bm, sync_out, sync_stride, tiles);
      else launch_vec<8, false>(grid, st, base, buf_stride, m, n_vec, stride, shadow, bm, sync_out, sync_stride, tiles);
    } else {
      if (BM) launch_vec<4, true>(grid, st, base, buf_stride, m, n_vec, stride, shadow, bm, sync_out, sync_stride, tiles);
      else launch_vec<4, false>(grid, st, base, buf_stride, m, n_vec, stride, shadow, bm, sync_out, sync_stride, tiles);
    }
    if (launches) ++*launches;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  const int64_t first = n_vec * W;
  if (first < n) {
    const int64_t gx = (n - first + kThreads - 1) / kThreads;
    if (gx > 2147483647LL) return cudaErrorInvalidValue;
    dim3 grid((unsigned)gx, (unsigned)n_buf);
    launch_dep(average_scalar_kernel, grid, dim3(kThreads), 0, st, 1, base, buf_stride, m, first, n, stride, shadow, bm,
               sync_out, sync_stride, tiles);
    if (launches) ++*launches;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

// pieces outside every blocked matrix (the bf16 copy has the master's element order there)
int launch_average_pieces(float* base, int n_buf, int64_t buf_stride, int m, const int64_t* begin, const int64_t* len,
                          int n_pieces, int64_t stride, __nv_bfloat16* shadow, cudaStream_t st, int64_t* launches,
                          float* sync_out, int64_t sync_stride) {
  if (n_pieces <= 0 || n_buf <= 0) return cudaSuccess;
  bool one = n_pieces <= kMaxPieces && aligned_to(base, 32) && stride % 8 == 0 && buf_stride % 8 == 0 &&
             aligned_to(shadow, 16) && aligned_to(sync_out, 32) && sync_stride % 8 == 0;
  for (int r = 0; r < n_pieces && one; ++r) one = begin[r] % 8 == 0 && len[r] % 8 == 0 && len[r] > 0;
  if (!one) {
    for (int r = 0; r < n_pieces; ++r) {
      int e = launch_average(base + begin[r], n_buf, buf_stride, m, len[r], stride, shadow ? shadow + begin[r] : nullptr, st,
                             launches, nullptr, sync_out ? sync_out + begin[r] : nullptr, sync_stride);
      if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
  }
  Pieces pc{};
  pc.n = n_pieces;
  for (int r = 0; r < n_pieces; ++r) {
    pc.begin[r] = begin[r];
    pc.first[r + 1] = pc.first[r] + len[r] / 8;
  }
  const int64_t gx = (pc.first[n_pieces] + kThreads - 1) / kThreads;
  if (gx > 2147483647LL) return cudaErrorInvalidValue;
  if (launches) ++*launches;
  return launch_dep(average_pieces_kernel, dim3((unsigned)gx, (unsigned)n_buf), dim3(kThreads), 0, st, 1, base, buf_stride, m,
                    pc, stride, shadow, sync_out, sync_stride);
}

}  // namespace ls

extern "C" int ls_average_flat(float* buf_dev, int m, int64_t P, int64_t stride, void* cuda_stream) {
  if (buf_dev == nullptr || m < 1 || P < 0 || stride < P) return LS_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(buf_dev) % 4 != 0) return LS_ERR_INVALID_ARG;
  int e = ls::launch_average(buf_dev, 1, 0, m, P, stride, nullptr, static_cast<cudaStream_t>(cuda_stream), nullptr,
                             nullptr, nullptr, 0, nullptr);
  return e == cudaSuccess ? LS_OK : LS_ERR_CUDA;
}

extern "C" int ls_block_average_flat(float* buf_dev, float* anchor_dev, float* u_dev, int m, int64_t P, int64_t stride,
                                     float lr, float beta, void* cuda_stream) {
  if (buf_dev == nullptr || anchor_dev == nullptr || u_dev == nullptr || m < 1 || P < 0 || stride < P)
    return LS_ERR_INVALID_ARG;
  if (!(lr > 0.f) || !isfinite(lr) || !(beta >= 0.f) || !isfinite(beta)) return LS_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(buf_dev) % 4 != 0 || reinterpret_cast<uintptr_t>(anchor_dev) % 4 != 0 ||
      reinterpret_cast<uintptr_t>(u_dev) % 4 != 0)
    return LS_ERR_INVALID_ARG;
  ls::BlockMomentum bm{anchor_dev, u_dev, lr, beta};
  int e = ls::launch_average(buf_dev, 1, 0, m, P, stride, nullptr, static_cast<cudaStream_t>(cuda_stream), nullptr,
                             &bm, nullptr, 0, nullptr);
  return e == cudaSuccess ? LS_OK : LS_ERR_CUDA;
}
