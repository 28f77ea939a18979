// Grouped matrix products on the 5th-generation tensor cores (tcgen05) with the
// layer arithmetic fused into the epilogue.  One CTA computes one 128 x BN
// output tile of one replica:
//
//   warp 0      TMA producer: cp.async.bulk.tensor tiles (128-byte swizzle) into a ring of stages
//   warp 1      allocates tensor memory, issues tcgen05.mma (one elected thread), accumulator in TMEM
//   warps 2-5   epilogue: tcgen05.ld the accumulator (warp w owns TMEM lanes 32*(w%4)..+31) and apply
//                 forward   Z = A W^T + b, relu, store as bf16            (evaluating f, Section 2)
//                 backward  dZ_prev = (dZ W) * 1[act > 0], store as bf16
//                 update    G = dZ^T A; v <- mu v + G; W <- W - eta v; refresh the bf16 copy of W
//                           (Section 2 mini-batch SGD update, Section 5.3 momentum); G never leaves the SM
//
// Operands are read in place whatever their orientation: a K-major operand
// ([rows][K], K contiguous) and an MN-major operand ([K][rows], rows contiguous)
// are both expressed through the shared-memory matrix descriptor, so no
// transposed copy of dZ, of the activations or of W is ever made.
//
// Every wait on an mbarrier is bounded; a wait that runs out records a code in
// *err_flag, and the CTA still frees its tensor memory and returns.
#include "ls_internal.h"
#include "tc_ptx.cuh"

namespace ls {
namespace {

using namespace ptx;

constexpr int BM = 128;            // rows of the output tile = TMEM lanes
constexpr int KB_BYTES = 128;      // bytes of K per stage row (one swizzle row)
constexpr int CHUNK_ROWS = 64;     // rows per TMA box
constexpr int CHUNK_BYTES = CHUNK_ROWS * KB_BYTES;   // 8 KB per TMA box
constexpr int kThreads = 192;
constexpr int kStageLd = 36;       // floats per staged row (32 + 4 padding) in the update epilogue

enum { EPI_FWD = 0, EPI_DX = 1, EPI_DW = 2 };

struct Operand {
  const int64_t* row_off;    // first row of group g (dataset rows), or null
  int64_t rows_per_group;    // else group g starts at row g*rows_per_group (2-D maps)
  int z0, z_step;            // 3-D maps: z = z0 + g*z_step
  int rank3;
};

struct Params {
  Operand a, b;
  int M, N, K;               // per group, in elements
  // forward
  const float* bias; int64_t bias_gstride; int relu;
  // forward / backward output, backward mask
  void* C; const void* act;
  // update
  float* W; float* V; __nv_bfloat16* Wb; int64_t w_gstride; float lr, mu;
  int* err_flag;
};

template <int BN, int STAGES, int EPI>
struct Smem {
  static constexpr int kStageBytes = BM * KB_BYTES + BN * KB_BYTES;
  // the update epilogue stages its 32x32 blocks in stage 0, which is free once the accumulator is complete
  static constexpr int kBarBytes = (2 * STAGES + 1) * 8 + 16;
  static constexpr int kTotal = 1024 + STAGES * kStageBytes + kBarBytes;
  static_assert(4 * 32 * kStageLd * 4 <= kStageBytes, "staging must fit in one stage");
};

__device__ __forceinline__ void issue_tile(void* dst, const CUtensorMap* tm, uint64_t* bar, const Operand& op, int g,
                                           bool mn_major, int tile0, int tile_extent, int k0, int elems_per_row) {
  // K-major: boxes of 64 rows, inner coordinate k0.  MN-major: boxes of 64 K-rows, inner coordinate = tile start.
  const int row_base = op.rank3 ? 0 : (int)(op.row_off ? op.row_off[g] : (int64_t)g * op.rows_per_group);
  const int z = op.z0 + g * op.z_step;
  if (!mn_major) {
    for (int r = 0; r < tile_extent / CHUNK_ROWS; ++r) {
      char* d = static_cast<char*>(dst) + r * CHUNK_BYTES;
      if (op.rank3) tma_load_3d(d, tm, bar, k0, tile0 + r * CHUNK_ROWS, z);
      else tma_load_2d(d, tm, bar, k0, row_base + tile0 + r * CHUNK_ROWS);
    }
  } else {
    for (int c = 0; c < tile_extent / elems_per_row; ++c) {
      char* d = static_cast<char*>(dst) + c * CHUNK_BYTES;
      if (op.rank3) tma_load_3d(d, tm, bar, tile0 + c * elems_per_row, k0, z);
      else tma_load_2d(d, tm, bar, tile0 + c * elems_per_row, row_base + k0);
    }
  }
}

__device__ __forceinline__ void store_bf16x8(__nv_bfloat16* p, const float* v) {
  uint4 u;
  __nv_bfloat162 t;
  t = __floats2bfloat162_rn(v[0], v[1]); u.x = *reinterpret_cast<uint32_t*>(&t);
  t = __floats2bfloat162_rn(v[2], v[3]); u.y = *reinterpret_cast<uint32_t*>(&t);
  t = __floats2bfloat162_rn(v[4], v[5]); u.z = *reinterpret_cast<uint32_t*>(&t);
  t = __floats2bfloat162_rn(v[6], v[7]); u.w = *reinterpret_cast<uint32_t*>(&t);
  *reinterpret_cast<uint4*>(p) = u;
}

template <int BN, bool A_MN, bool B_MN, int EPI, int STAGES>
__global__ void __launch_bounds__(kThreads, (Smem<BN, STAGES, EPI>::kTotal <= 113 * 1024) ? 2 : 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const Params p) {
  using L = Smem<BN, STAGES, EPI>;
  constexpr int ELEMS = KB_BYTES / 2;          // bf16 elements per 128-byte row = K elements per stage
  constexpr int MMA_K = 16;                    // K of one tcgen05.mma, bf16
  constexpr uint32_t IDESC = make_idesc(1u /*bf16*/, A_MN, B_MN, BM, BN);

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* stage_base = smem;
  float* staging = reinterpret_cast<float*>(smem);
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + STAGES * L::kStageBytes);
  uint64_t* empty = full + STAGES;
  uint64_t* accum = empty + STAGES;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(accum + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = blockIdx.z;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  const int num_kb = p.K / ELEMS;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(accum, 1);
    fence_mbar_init();
    prefetch_tmap(&tmA);
    prefetch_tmap(&tmB);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, BN);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (elect_one()) {
      for (int kb = 0; kb < num_kb; ++kb) {
        const int s = kb % STAGES;
        if (kb >= STAGES && !mbar_wait(&empty[s], ((kb / STAGES) - 1) & 1)) { atomicExch(p.err_flag, 1); break; }
        mbar_expect_tx(&full[s], L::kStageBytes);
        uint8_t* sa = stage_base + s * L::kStageBytes;
        uint8_t* sb = sa + BM * KB_BYTES;
        issue_tile(sa, &tmA, &full[s], p.a, g, A_MN, m0, BM, kb * ELEMS, ELEMS);
        issue_tile(sb, &tmB, &full[s], p.b, g, B_MN, n0, BN, kb * ELEMS, ELEMS);
      }
    }
  } else if (warp == 1) {
    if (elect_one()) {
      bool ok = true;
      for (int kb = 0; kb < num_kb && ok; ++kb) {
        const int s = kb % STAGES;
        if (!mbar_wait(&full[s], (kb / STAGES) & 1)) { atomicExch(p.err_flag, 2); ok = false; break; }
        tc_fence_after_sync();
        const uint32_t a_addr = smem_u32(stage_base + s * L::kStageBytes);
        const uint32_t b_addr = a_addr + BM * KB_BYTES;
#pragma unroll
        for (int k = 0; k < ELEMS / MMA_K; ++k) {
          // K-major: the next 16 elements of K are 32 bytes further along each swizzled row.
          // MN-major: they are the next 16 K-rows (16 x 128 bytes); chunks of 64 rows-of-MN follow every 8 KB.
          const uint64_t da = A_MN ? make_smem_desc(a_addr + k * MMA_K * KB_BYTES, CHUNK_BYTES, 1024)
                                   : make_smem_desc(a_addr + k * MMA_K * 2, 16, 1024);
          const uint64_t db = B_MN ? make_smem_desc(b_addr + k * MMA_K * KB_BYTES, CHUNK_BYTES, 1024)
                                   : make_smem_desc(b_addr + k * MMA_K * 2, 16, 1024);
          mma_bf16(tmem_base, da, db, IDESC, (kb | k) != 0 ? 1u : 0u);
        }
        mma_commit(&empty[s]);     // frees the stage once these MMAs have read it
      }
      mma_commit(accum);           // accumulator complete
    }
  } else {
    // ---- epilogue warps ---------------------------------------------------------
    const int q = warp & 3;
    const int row = m0 + q * 32 + lane;        // output row this thread owns
    bool ok = mbar_wait(accum, 0);
    if (!ok && lane == 0) atomicExch(p.err_flag, 3);
    ok = __all_sync(0xffffffffu, ok);
    tc_fence_after_sync();
    if (ok) {
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
      for (int c = 0; c < BN / 32; ++c) {
        uint32_t r[32];
        tmem_ld_32x32(taddr + c * 32, r);
        tmem_ld_wait();
        const int col = n0 + c * 32;
        if (EPI == EPI_FWD) {
          float o[32];
          const float* bias = p.bias ? p.bias + (int64_t)g * p.bias_gstride + col : nullptr;
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            float v = __uint_as_float(r[i]);
            if (bias) v += __ldg(bias + i);
            o[i] = (p.relu && !(v > 0.f)) ? 0.f : v;
          }
          __nv_bfloat16* out = static_cast<__nv_bfloat16*>(p.C) + ((int64_t)g * p.M + row) * p.N + col;
#pragma unroll
          for (int i = 0; i < 4; ++i) store_bf16x8(out + i * 8, o + i * 8);
        } else if (EPI == EPI_DX) {
          const int64_t at = ((int64_t)g * p.M + row) * p.N + col;
          const uint4* a4 = reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(p.act) + at);
          float o[32];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const uint4 u = a4[i];
            const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              // a bf16 is positive iff it is non-zero with the sign bit clear
              const uint32_t lo = w[j] & 0xFFFFu, hi = w[j] >> 16;
              o[i * 8 + j * 2] = (lo != 0 && lo < 0x8000u) ? __uint_as_float(r[i * 8 + j * 2]) : 0.f;
              o[i * 8 + j * 2 + 1] = (hi != 0 && hi < 0x8000u) ? __uint_as_float(r[i * 8 + j * 2 + 1]) : 0.f;
            }
          }
          __nv_bfloat16* out = static_cast<__nv_bfloat16*>(p.C) + at;
#pragma unroll
          for (int i = 0; i < 4; ++i) store_bf16x8(out + i * 8, o + i * 8);
        } else {
          // transpose the 32x32 block through shared memory so that global accesses run along rows
          float* st = staging + (warp - 2) * 32 * kStageLd;
#pragma unroll
          for (int i = 0; i < 8; ++i)
            *reinterpret_cast<float4*>(&st[lane * kStageLd + i * 4]) =
                make_float4(__uint_as_float(r[4 * i]), __uint_as_float(r[4 * i + 1]), __uint_as_float(r[4 * i + 2]),
                            __uint_as_float(r[4 * i + 3]));
          __syncwarp();
          const int cc = (lane & 7) * 4;
          // all 16 row-segment loads of this block are issued before the first use
          float4 w4[8], v4[8];
          const int64_t at0 = (int64_t)g * p.w_gstride + (int64_t)(m0 + q * 32 + (lane >> 3)) * p.N + col + cc;
#pragma unroll
          for (int it = 0; it < 8; ++it) {
            const int64_t at = at0 + (int64_t)(it * 4) * p.N;
            w4[it] = *reinterpret_cast<const float4*>(p.W + at);
            if (p.mu != 0.f) v4[it] = *reinterpret_cast<const float4*>(p.V + at);
          }
#pragma unroll
          for (int it = 0; it < 8; ++it) {
            const int rr = it * 4 + (lane >> 3);
            const int64_t at = at0 + (int64_t)(it * 4) * p.N;
            const float4 gacc = *reinterpret_cast<const float4*>(&st[rr * kStageLd + cc]);
            float gs[4] = {gacc.x, gacc.y, gacc.z, gacc.w};
            float ws[4] = {w4[it].x, w4[it].y, w4[it].z, w4[it].w};
            float vs[4] = {0.f, 0.f, 0.f, 0.f};
            if (p.mu != 0.f) { vs[0] = v4[it].x; vs[1] = v4[it].y; vs[2] = v4[it].z; vs[3] = v4[it].w; }
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float step = (p.mu != 0.f) ? fmaf(p.mu, vs[e], gs[e]) : gs[e];
              vs[e] = step;
              ws[e] = fmaf(-p.lr, step, ws[e]);
            }
            *reinterpret_cast<float4*>(p.W + at) = make_float4(ws[0], ws[1], ws[2], ws[3]);
            if (p.mu != 0.f) *reinterpret_cast<float4*>(p.V + at) = make_float4(vs[0], vs[1], vs[2], vs[3]);
            if (p.Wb != nullptr) {
              __nv_bfloat162 lo = __floats2bfloat162_rn(ws[0], ws[1]);
              __nv_bfloat162 hi = __floats2bfloat162_rn(ws[2], ws[3]);
              uint2 u;
              u.x = *reinterpret_cast<uint32_t*>(&lo);
              u.y = *reinterpret_cast<uint32_t*>(&hi);
              *reinterpret_cast<uint2*>(p.Wb + at) = u;
            }
          }
          __syncwarp();
        }
      }
    }
    tc_fence_before_sync();
  }
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, BN);
  }
}

// ---- host side -----------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) == cudaSuccess &&
        qr == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

template <int BN, bool A_MN, bool B_MN, int EPI, int STAGES>
int launch_one(const CUtensorMap& a, const CUtensorMap& b, const Params& p, int groups, cudaStream_t st) {
  using L = Smem<BN, STAGES, EPI>;
  auto kern = tc_gemm_kernel<BN, A_MN, B_MN, EPI, STAGES>;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kTotal);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  dim3 grid((unsigned)(p.N / BN), (unsigned)(p.M / BM), (unsigned)groups);
  kern<<<grid, kThreads, L::kTotal, st>>>(a, b, p);
  return cudaGetLastError();
}

}  // namespace

// 2-D map over a row-major bf16 matrix [rows][cols], box 64 x 64, 128-byte swizzle.
int tc_make_map_2d(CUtensorMap* out, const void* base, int64_t rows, int64_t cols) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return cudaErrorNotSupported;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {64, 64};
  cuuint32_t es[2] = {1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, es,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

// 3-D map over `groups` row-major bf16 matrices [rows][cols] that start every gstride elements.
int tc_make_map_3d(CUtensorMap* out, const void* base, int64_t rows, int64_t cols, int64_t groups, int64_t gstride) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return cudaErrorNotSupported;
  cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)groups};
  cuuint64_t strides[2] = {(cuuint64_t)cols * 2, (cuuint64_t)gstride * 2};
  cuuint32_t box[3] = {64, 64, 1};
  cuuint32_t es[3] = {1, 1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, es,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

bool tc_shape_ok(int M, int N, int K) { return M % BM == 0 && N % 128 == 0 && K % 64 == 0 && M > 0 && N > 0 && K > 0; }

int launch_tc_fwd(const TcFwdArgs& a, cudaStream_t st, int64_t* launches) {
  Params p{};
  p.a = Operand{a.row_off, a.M, 0, 0, 0};
  p.b = Operand{nullptr, 0, a.w_z0, a.w_zstep, 1};
  p.M = a.M; p.N = a.N; p.K = a.K;
  p.bias = a.bias; p.bias_gstride = a.bias_gstride; p.relu = a.relu;
  p.C = a.C; p.err_flag = a.err_flag;
  if (launches) ++*launches;
  if (a.N % 256 == 0) return launch_one<256, false, false, EPI_FWD, 4>(*a.mapA, *a.mapW, p, a.groups, st);
  return launch_one<128, false, false, EPI_FWD, 4>(*a.mapA, *a.mapW, p, a.groups, st);
}

int launch_tc_dx(const TcDxArgs& a, cudaStream_t st, int64_t* launches) {
  Params p{};
  p.a = Operand{nullptr, a.M, 0, 0, 0};
  p.b = Operand{nullptr, 0, 0, 1, 1};
  p.M = a.M; p.N = a.N; p.K = a.K;
  p.C = a.C; p.act = a.act; p.err_flag = a.err_flag;
  if (launches) ++*launches;
  if (a.N % 256 == 0) return launch_one<256, false, true, EPI_DX, 4>(*a.mapDz, *a.mapW, p, a.groups, st);
  return launch_one<128, false, true, EPI_DX, 4>(*a.mapDz, *a.mapW, p, a.groups, st);
}

int launch_tc_dw(const TcDwArgs& a, cudaStream_t st, int64_t* launches) {
  Params p{};
  p.a = Operand{nullptr, a.B, 0, 0, 0};
  p.b = Operand{a.row_off, a.B, 0, 0, 0};
  p.M = a.M; p.N = a.N; p.K = a.B;
  p.W = a.W; p.V = a.V; p.Wb = a.Wb; p.w_gstride = a.w_gstride; p.lr = a.lr; p.mu = a.mu;
  p.err_flag = a.err_flag;
  if (launches) ++*launches;
  return launch_one<128, true, true, EPI_DW, 3>(*a.mapDz, *a.mapA, p, a.groups, st);
}

}  // namespace ls
