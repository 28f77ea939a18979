// Grouped matrix products on the 5th-generation tensor cores (tcgen05) with the
// layer arithmetic fused into the epilogue.  One CTA computes one 128 x BN
// output tile of one replica:
//
//   warp 0      TMA producer: cp.async.bulk.tensor tiles (128-byte swizzle) into a ring of stages
//   warp 1      allocates tensor memory, issues tcgen05.mma (one elected thread), accumulator in TMEM
//   warps 2-5   epilogue: tcgen05.ld the accumulator (warp w owns TMEM lanes 32*(w%4)..+31) and apply
//                 forward   Z = A W^T + b, relu                            (evaluating f, Section 2);
//                           when the next layer is the narrow output layer and the tile holds the whole
//                           mini-batch, also that layer: partial logits of this CTA's columns go to a
//                           scratch, and the last CTA of the replica to finish adds them in a fixed
//                           order and forms the per-sample losses and dZ of the output layer
//                 backward  dZ_prev = (dZ W) * 1[act > 0]; when the tile holds the whole mini-batch, also the
//                           bias update of the layer below from the column sums of dZ_prev
//                 update    G = dZ^T A; v <- mu v + G; W <- W - eta v      (Section 2 mini-batch SGD
//                           update, Section 5.3 momentum); G never leaves the SM
//
// Two operand formats:
//   bf16   one tcgen05.mma kind::f16 per 16 elements of K; outputs rounded to bf16.
//   fp32   every fp32 operand x is used as the pair (hi, lo): hi is x itself, of which the tensor
//          core reads the upper 19 bits (tf32); lo = x - tf32(x) is written by two splitter warps
//          (warps 6-7) from each stage that TMA has filled into a second, shorter ring of shared
//          memory, in the same (swizzled) layout.  Three kind::tf32 MMAs per 8 elements of K
//          (lo*hi + hi*lo + hi*hi) give products accurate to about 2^-21, accumulated in fp32.
//          The tensor core's fp32 accumulation truncates, which biases a long sum; the forward and
//          backward kernels therefore restart the TMEM accumulator every kChunkStages stages (two
//          accumulators, double-buffered) and the epilogue warps add the partial sums in registers
//          with round-to-nearest while the next chunk is being multiplied.
//          When a layer has too few output tiles to occupy the GPU (small batch x width), K is split
//          over a thread-block cluster of 2 or 4 CTAs: every CTA sums its K slice as above and leaves
//          its partial tile in shared memory; then CTA r adds, in rank order, the partial sums of
//          columns [r BN/S, (r+1) BN/S) through distributed shared memory and runs the epilogue for
//          them (a reduce-scatter).  No atomics, so the result is reproducible.
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
constexpr int kThreadsBf16 = 192;  // warps 0-5
constexpr int kSplitWarps = 4;
constexpr int kThreadsFp32 = 192 + 32 * kSplitWarps;  // + the splitter warps
constexpr int kHeadMax = 16;       // outputs of a fused narrow output layer, at most
constexpr int kStageLd = 36;       // floats per staged row (32 + 4 padding) in the update epilogue
constexpr int kChunkStages = 4;    // fp32 forward/backward: stages per TMEM accumulation chunk (48 MMAs)

enum { EPI_FWD = 0, EPI_DX = 1, EPI_DW = 2 };

struct Operand {
  const int64_t* row_off;    // first row of group g (dataset rows), or null
  int64_t rows_per_group;    // else group g starts at row g*rows_per_group (2-D maps)
  int z0, z_step;            // 3-D maps: z = z0 + g*z_step
  int rank3;                 // 0: 2-D map; 1: 3-D map [group][row][column]; 2: panel map [group][column / 64][row][64]
};

struct Params {
  Operand a, b;
  int M, N, K;               // per group, in elements
  // forward
  const float* bias; int64_t bias_gstride; int relu;
  // forward / backward output, backward mask
  void* C; const void* act;
  // backward: bias of the layer below and its momentum (or null), elements between replicas
  float* dbias; float* dvbias; int64_t dbias_gstride;
  // forward: the narrow output layer that follows (hW null: none)
  TcHead head;
  // update
  float* W; float* V; __nv_bfloat16* Wb; int64_t w_gstride; float lr, mu;
  int* err_flag;
};

// Shared memory: a ring of STAGES stages filled by TMA (the A and B tiles as they are in memory) and,
// for fp32 operands, a shorter ring of kLoStages stages that receives their lo parts.
template <bool TF32, int BN, int STAGES, int MT = 1>
struct Smem {
  static constexpr int kLoStages = TF32 ? 2 : 0;
  static constexpr int kABytes = MT * BM * KB_BYTES;   // MT row blocks of 128 share one B tile
  static constexpr int kBBytes = BN * KB_BYTES;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kRingBytes = (STAGES + kLoStages) * kStageBytes;
  // the update epilogue stages its 32x32 blocks in stage 0, which is free once the accumulator is complete
  static constexpr int kBarBytes = (2 * STAGES + 2 * 2 + 4) * 8 + 16;
  static constexpr int kTotal = 1024 + kRingBytes + kBarBytes;
  static_assert(4 * 32 * kStageLd * 4 <= kStageBytes, "staging must fit in one stage");
  static_assert((4 * 32 * kStageLd + MT * 4 * BN) * 4 <= kRingBytes, "column-sum scratch of the backward epilogue");
  static_assert(kTotal <= 227 * 1024, "shared memory budget");
};

__device__ __forceinline__ int operand_row_base(const Operand& op, int g) {
  return op.rank3 ? 0 : (int)(op.row_off ? op.row_off[g] : (int64_t)g * op.rows_per_group);
}
// Bring one operand tile of `tile_extent` MN-rows x ELEMS K-elements into shared memory as boxes of
// 128 bytes x ELEMS rows.  K-major: box rows are MN-rows, inner coordinate k0.  MN-major: box rows are
// K-rows, inner coordinate is the tile start; chunks of ELEMS MN-elements follow each other.
// row_base = operand_row_base(op, g), read once by the caller (for dataset rows it is a global load).
template <int ELEMS>
__device__ __forceinline__ void issue_tile(void* dst, const CUtensorMap* tm, uint64_t* bar, const Operand& op, int g,
                                           int row_base, bool mn_major, int tile0, int tile_extent, int k0,
                                           uint64_t pol) {
  // rows per box: a K-major box always holds 64 MN-rows, an MN-major box holds ELEMS K-rows
  const int box_rows = mn_major ? ELEMS : 64;
  const int kChunkBytes = box_rows * KB_BYTES;
  const int z = op.z0 + g * op.z_step;
  const int n_boxes = mn_major ? tile_extent / ELEMS : tile_extent / 64;
  for (int c = 0; c < n_boxes; ++c) {
    char* d = static_cast<char*>(dst) + c * kChunkBytes;
    const int x = mn_major ? tile0 + c * ELEMS : k0;
    const int y = mn_major ? k0 : tile0 + c * 64;
    if (op.rank3 == 2) tma_load_4d_hint(d, tm, bar, 0, y, x >> 6, z, pol);     // x is a multiple of 64
    else if (op.rank3) tma_load_3d_hint(d, tm, bar, x, y, z, pol);
    else tma_load_2d_hint(d, tm, bar, x, row_base + y, pol);
  }
}

// one 32-byte (whole sector) store; p must be 32-byte aligned
__device__ __forceinline__ void st_global_v8(void* p, const uint32_t (&v)[8]) {
  asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]),
               "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
               : "memory");
}

// Store 32 consecutive outputs of one row (bf16 or fp32) in whole 32-byte sectors.
template <bool TF32>
__device__ __forceinline__ void store_row32(void* C, int64_t at, const float (&o)[32]) {
  if (TF32) {
    float* c = static_cast<float*>(C) + at;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      uint32_t hi[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) hi[e] = __float_as_uint(o[8 * i + e]);
      st_global_v8(c + 8 * i, hi);
    }
  } else {
    __nv_bfloat16* out = static_cast<__nv_bfloat16*>(C) + at;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      uint32_t u[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        __nv_bfloat162 t = __floats2bfloat162_rn(o[16 * i + 2 * e], o[16 * i + 2 * e + 1]);
        u[e] = *reinterpret_cast<uint32_t*>(&t);
      }
      st_global_v8(out + 16 * i, u);
    }
  }
}

// MT = 2: the CTA computes two 128-row blocks (a 256 x BN tile) from one B tile in shared memory, with two
// TMEM accumulators: a third less operand traffic from L2 per flop, which is what bounds these kernels.
template <bool TF32, int BN, bool A_MN, bool B_MN, int EPI, int STAGES, int SPLIT, int MT>
__global__ void __launch_bounds__(TF32 ? kThreadsFp32 : kThreadsBf16, (Smem<TF32, BN, STAGES, MT>::kTotal <= 113 * 1024) ? 2 : 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const Params p) {
  using L = Smem<TF32, BN, STAGES, MT>;
  constexpr int EB = TF32 ? 4 : 2;             // bytes per operand element
  constexpr int ELEMS = KB_BYTES / EB;         // K elements per stage
  constexpr int MMA_K = 32 / EB;               // K of one tcgen05.mma (32 bytes)
  constexpr int CHUNK_BYTES = ELEMS * KB_BYTES;
  constexpr uint32_t IDESC = make_idesc(TF32 ? 2u : 1u, A_MN, B_MN, BM, BN);
  constexpr bool CHUNKED = TF32 && EPI != EPI_DW;
  constexpr int CS = kChunkStages;
  constexpr uint32_t TMEM_COLS = CHUNKED ? 2 * BN : MT * BN;
  static_assert(MT == 1 || (!CHUNKED && !A_MN && EPI != EPI_DW && MT * BN <= 512), "two row blocks: bf16 forward/backward");
  static_assert(SPLIT == 1 || CHUNKED, "split-K needs the register-resident partial sums");
  static_assert(SPLIT == 1 || BN * BM * 4 <= L::kRingBytes, "exchange buffer");
  constexpr int CPR = BN / SPLIT;              // columns that each CTA of the cluster finishes
  static_assert(CPR % 32 == 0, "whole 32-column blocks per CTA");

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* stage_base = smem;
  float* staging = reinterpret_cast<float*>(smem);
  float* colsum = staging + 4 * 32 * kStageLd;      // [MT * 4][BN] partial column sums (backward epilogue)
  uint8_t* lo_base = smem + STAGES * L::kStageBytes;
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + L::kRingBytes);
  uint64_t* empty = full + STAGES;
  uint64_t* acc_full = empty + STAGES;      // [2] accumulator (chunk) complete
  uint64_t* acc_empty = acc_full + 2;        // [2] accumulator drained by the 4 epilogue warps
  uint64_t* lo_full = acc_empty + 2;         // [2] fp32: lo parts of a stage written
  uint64_t* lo_empty = lo_full + 2;          // [2] ... and read by the tensor core
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(lo_empty + 2);
  constexpr int LS = L::kLoStages > 0 ? L::kLoStages : 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = blockIdx.z;
  const int m0 = blockIdx.y * BM * MT, n0 = (int)(blockIdx.x / SPLIT) * BN;
  const int rank = SPLIT > 1 ? (int)cluster_ctarank() : 0;     // which K slice this CTA sums
  const int num_kb = p.K / ELEMS / SPLIT;
  const int kb0 = rank * num_kb;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 4);
      mbar_init(&lo_full[b], kSplitWarps); mbar_init(&lo_empty[b], 1);
    }
    fence_mbar_init();
    prefetch_tmap(&tmA);
    prefetch_tmap(&tmB);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  grid_dep_wait();        // everything above overlapped the previous kernel; its results are needed from here on
  grid_dep_launch();

  // epilogue-warp state (warps 2-5): this thread owns output row `row`
  const int q = warp & 3;
  const int row0 = m0 + q * 32 + lane;
  const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
  float sum[CHUNKED ? BN : 1];
  bool ok = true;
  // fused output layer: its weights for this CTA's columns ([class][CPR], as float4) and this thread's
  // labels are requested now and parked in registers until the stage memory is free
  constexpr int HP = (EPI == EPI_FWD) ? (kHeadMax * CPR / 4 + 127) / 128 : 1;
  float4 hw_pref[HP];
  int h_label[EPI == EPI_FWD ? MT : 1];
  float h_target[EPI == EPI_FWD ? MT : 1];
  if (EPI == EPI_FWD && warp >= 2 && warp < 6 && p.head.W != nullptr) {
    const float* hw = p.head.W + (int64_t)g * p.head.w_gstride + n0 + rank * CPR;
#pragma unroll
    for (int i = 0; i < HP; ++i) {
      const int idx = (int)threadIdx.x - 64 + i * 128;
      const int cls = idx / (CPR / 4), c4 = idx % (CPR / 4);
      hw_pref[i] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (cls < p.head.C) hw_pref[i] = __ldg(reinterpret_cast<const float4*>(hw + (int64_t)cls * p.N) + c4);
    }
    const int64_t y0 = p.head.y_row_off[g];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      h_label[mt] = 0; h_target[mt] = 0.f;
      if (p.head.kind == LS_LOSS_SOFTMAX_CE) h_label[mt] = static_cast<const int32_t*>(p.head.y)[y0 + mt * BM + q * 32 + lane];
      else h_target[mt] = static_cast<const float*>(p.head.y)[y0 + mt * BM + q * 32 + lane];
    }
  }

  if (warp == 0) {
    if (elect_one()) {
      // the A tile (activations, gradients) is re-read by every CTA of its replica, the weight tile by nobody:
      // L2 keeps the former and lets the latter go first
      const uint64_t pol_a = l2_policy(2), pol_b = l2_policy(EPI == EPI_DW ? 2 : 1);
      const int a_base = operand_row_base(p.a, g), b_base = operand_row_base(p.b, g);
      for (int kb = 0; kb < num_kb; ++kb) {
        const int s = kb % STAGES;
        if (kb >= STAGES && !mbar_wait(&empty[s], ((kb / STAGES) - 1) & 1)) { atomicExch(p.err_flag, 1); break; }
        mbar_expect_tx(&full[s], L::kStageBytes);
        uint8_t* sa = stage_base + s * L::kStageBytes;
        uint8_t* sb = sa + L::kABytes;
        const int k0 = (kb0 + kb) * ELEMS;
        issue_tile<ELEMS>(sa, &tmA, &full[s], p.a, g, a_base, A_MN, m0, BM * MT, k0, pol_a);
        issue_tile<ELEMS>(sb, &tmB, &full[s], p.b, g, b_base, B_MN, n0, BN, k0, pol_b);
      }
    }
  } else if (TF32 && warp >= 6) {
    // ---- splitter warps (fp32): lo = x - tf32(x) of both tiles of the stage, element by element, so
    // the copy has the layout (swizzle included) of the tile it comes from
    const int tid = threadIdx.x - 6 * 32;
    for (int kb = 0; kb < num_kb; ++kb) {
      const int s = kb % STAGES, sl = kb % LS;
      bool got = mbar_wait(&full[s], (kb / STAGES) & 1);
      if (got && kb >= LS) got = mbar_wait(&lo_empty[sl], ((kb / LS) - 1) & 1);
      if (!__all_sync(0xffffffffu, got)) {
        if (lane == 0) atomicExch(p.err_flag, 5);
        break;
      }
      constexpr int kSplitDepth = (L::kStageBytes % (8 * 16 * kSplitWarps * 32) == 0) ? 8 : 4;
      static_assert(L::kStageBytes % (kSplitDepth * 16 * kSplitWarps * 32) == 0, "whole batches of pieces");
      split_lo_smem<kSplitDepth>(smem_u32(stage_base + s * L::kStageBytes), smem_u32(lo_base + sl * L::kStageBytes),
                                 L::kStageBytes, tid, kSplitWarps * 32);
      fence_proxy_async_smem();     // the tensor core reads shared memory through the async proxy
      __syncwarp();
      if (lane == 0) mbar_arrive(&lo_full[sl]);
    }
  } else if (warp == 1) {
    if (elect_one()) {
      for (int kb = 0; kb < num_kb; ++kb) {
        const int s = kb % STAGES;
        const int chunk = CHUNKED ? kb / CS : 0;
        const uint32_t d_tmem = tmem_base + (uint32_t)((chunk & 1) * BN);
        const bool chunk_start = CHUNKED ? (kb % CS == 0) : (kb == 0);
        if (CHUNKED && chunk_start && chunk >= 2 && !mbar_wait(&acc_empty[chunk & 1], ((chunk >> 1) - 1) & 1)) {
          atomicExch(p.err_flag, 4);
          break;
        }
        if (!mbar_wait(&full[s], (kb / STAGES) & 1)) { atomicExch(p.err_flag, 2); break; }
        if (TF32 && !mbar_wait(&lo_full[kb % LS], (kb / LS) & 1)) { atomicExch(p.err_flag, 6); break; }
        tc_fence_after_sync();
        const uint32_t a_addr = smem_u32(stage_base + s * L::kStageBytes);
        const uint32_t b_addr = a_addr + L::kABytes;
        const uint32_t alo_addr = smem_u32(lo_base + (kb % LS) * L::kStageBytes);
        const uint32_t blo_addr = alo_addr + L::kABytes;
#pragma unroll
        for (int k = 0; k < ELEMS / MMA_K; ++k) {
          // K-major: the next MMA_K elements of K are 32 bytes further along each swizzled row.
          // MN-major: they are the next MMA_K K-rows of 128 bytes; chunks of MN follow every CHUNK_BYTES.
          const uint32_t a_adv = A_MN ? k * MMA_K * KB_BYTES : k * 32;
          const uint32_t b_adv = B_MN ? k * MMA_K * KB_BYTES : k * 32;
          // An MN-major operand of 32-bit elements must use the 128-byte swizzle with 32-byte units,
          // whose period is 4 K-rows (512 bytes); everything else uses 16-byte units, period 8 rows.
          const uint32_t a_lbo = A_MN ? CHUNK_BYTES : 16, b_lbo = B_MN ? CHUNK_BYTES : 16;
          const uint32_t a_sw = (TF32 && A_MN) ? kSwizzle128B_32B : kSwizzle128B;
          const uint32_t b_sw = (TF32 && B_MN) ? kSwizzle128B_32B : kSwizzle128B;
          const uint32_t a_sbo = (TF32 && A_MN) ? 512 : 1024, b_sbo = (TF32 && B_MN) ? 512 : 1024;
          const uint64_t da = make_smem_desc(a_addr + a_adv, a_lbo, a_sbo, a_sw);
          const uint64_t db = make_smem_desc(b_addr + b_adv, b_lbo, b_sbo, b_sw);
          if (TF32) {
            const uint64_t dal = make_smem_desc(alo_addr + a_adv, a_lbo, a_sbo, a_sw);
            const uint64_t dbl = make_smem_desc(blo_addr + b_adv, b_lbo, b_sbo, b_sw);
            mma_tf32(d_tmem, dal, db, IDESC, (chunk_start && k == 0) ? 0u : 1u);
            mma_tf32(d_tmem, da, dbl, IDESC, 1u);
            mma_tf32(d_tmem, da, db, IDESC, 1u);
          } else {
            mma_bf16(d_tmem, da, db, IDESC, (chunk_start && k == 0) ? 0u : 1u);
            if (MT == 2) {
              // second row block: same B tile, A rows 128..255 (16 KB further in the stage)
              const uint64_t da2 = make_smem_desc(a_addr + BM * KB_BYTES + a_adv, a_lbo, a_sbo, a_sw);
              mma_bf16(d_tmem + BN, da2, db, IDESC, (chunk_start && k == 0) ? 0u : 1u);
            }
          }
        }
        mma_commit(&empty[s]);     // frees the stage once these MMAs have read it
        if (TF32) mma_commit(&lo_empty[kb % LS]);
        if (CHUNKED ? (kb % CS == CS - 1 || kb == num_kb - 1) : (kb == num_kb - 1))
          mma_commit(&acc_full[chunk & 1]);     // this accumulator is complete
      }
    }
  } else if (warp < 6) {
    // ---- epilogue warps: collect the accumulator(s) ------------------------------
    if (CHUNKED) {
      // add the partial accumulators in registers (this thread owns one output row) as they complete
#pragma unroll
      for (int i = 0; i < BN; ++i) sum[i] = 0.f;
      const int num_chunks = (num_kb + CS - 1) / CS;
      for (int ch = 0; ch < num_chunks && ok; ++ch) {
        const int buf = ch & 1;
        ok = mbar_wait(&acc_full[buf], (ch >> 1) & 1);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after_sync();
#pragma unroll
        for (int c = 0; c < BN / 32; ++c) {
          uint32_t r[32];
          tmem_ld_32x32(taddr + buf * BN + c * 32, r);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) sum[c * 32 + i] += __uint_as_float(r[i]);
        }
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(&acc_empty[buf]);
      }
    } else {
      ok = mbar_wait(&acc_full[0], 0);
      ok = __all_sync(0xffffffffu, ok);
      tc_fence_after_sync();
    }
    if (!ok && lane == 0) atomicExch(p.err_flag, 3);
    if (SPLIT > 1 && ok) {
      // every load of this CTA has been consumed and every MMA has completed: the stage buffers are
      // free, and hold this CTA's partial tile for the cluster ([column][row], so lanes are conflict-free)
      float* xbuf = reinterpret_cast<float*>(smem);
#pragma unroll
      for (int i = 0; i < (CHUNKED ? BN : 1); ++i) xbuf[i * BM + q * 32 + lane] = sum[i];
    }
  }
  if (SPLIT > 1) {
    cluster_sync_all();
    if (warp >= 2 && warp < 6 && ok) {
      // this CTA's columns, added in rank order whoever adds them
      const uint32_t mine = smem_u32(reinterpret_cast<float*>(smem) + (rank * CPR) * BM + q * 32 + lane);
#pragma unroll
      for (int r = 0; r < SPLIT; ++r) {
        const uint32_t remote = map_to_rank(mine, (uint32_t)r);
#pragma unroll
        for (int i = 0; i < (CHUNKED ? CPR : 1); ++i) {
          const float v = ld_cluster_f32(remote + (uint32_t)(i * BM * 4));
          sum[i] = (r == 0) ? v : sum[i] + v;
        }
      }
    }
    cluster_sync_all();      // every CTA stays alive until the others have read its tile
  }
  if (warp >= 2 && warp < 6) {
    // weights of the fused output layer: behind the exchange tile, which other CTAs may still be reading
    float4* ws4 = reinterpret_cast<float4*>(smem + (SPLIT > 1 ? BN * BM * 4 : 0) + 256);
    if (EPI == EPI_FWD && p.head.W != nullptr) {
#pragma unroll
      for (int i = 0; i < HP; ++i) {
        const int idx = (int)threadIdx.x - 64 + i * 128;
        if (idx < kHeadMax * CPR / 4) ws4[idx] = hw_pref[i];
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
    }
    float hl[EPI == EPI_FWD ? MT : 1][kHeadMax];      // partial logits of this thread's row(s)
#pragma unroll
    for (int i = 0; i < (EPI == EPI_FWD ? MT : 1); ++i)
#pragma unroll
      for (int cls = 0; cls < kHeadMax; ++cls) hl[i][cls] = 0.f;
    if (ok) {
#pragma unroll
      for (int cc32 = 0; cc32 < MT * (CPR / 32); ++cc32) {
        const int mt = cc32 / (CPR / 32), c = cc32 % (CPR / 32);
        const int row = row0 + mt * BM;          // output row this thread owns in row block mt
        uint32_t r[32];
        if (CHUNKED) {
#pragma unroll
          for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(sum[c * 32 + i]);
        } else {
          tmem_ld_32x32(taddr + mt * BN + c * 32, r);
          tmem_ld_wait();
        }
        const int col = n0 + rank * CPR + c * 32;
        if (EPI == EPI_FWD) {
          float o[32];
          const float* bias = p.bias ? p.bias + (int64_t)g * p.bias_gstride + col : nullptr;
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            float v = __uint_as_float(r[i]);
            if (bias) v += __ldg(bias + i);
            o[i] = (p.relu && !(v > 0.f)) ? 0.f : v;
          }
          store_row32<TF32>(p.C, ((int64_t)g * p.M + row) * p.N + col, o);
          if (p.head.W != nullptr) {
            // logits of the output layer restricted to these 32 columns (of the values as stored)
            if (!TF32) {
#pragma unroll
              for (int i = 0; i < 32; ++i) o[i] = __bfloat162float(__float2bfloat16_rn(o[i]));
            }
#pragma unroll
            for (int cls = 0; cls < kHeadMax; ++cls) {
              if (cls < p.head.C) {           // uniform; the classes are independent chains
                const float4* w4 = ws4 + (cls * CPR + c * 32) / 4;
                float a = 0.f;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                  const float4 w = w4[i];
                  a = fmaf(o[4 * i + 3], w.w, fmaf(o[4 * i + 2], w.z, fmaf(o[4 * i + 1], w.y, fmaf(o[4 * i], w.x, a))));
                }
                hl[mt][cls] += a;
              }
            }
          }
        } else if (EPI == EPI_DX) {
          const int64_t at = ((int64_t)g * p.M + row) * p.N + col;
          float o[32];
          if (TF32) {
            const float4* a4 = reinterpret_cast<const float4*>(static_cast<const float*>(p.act) + at);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const float4 a = a4[i];
              o[4 * i] = a.x > 0.f ? __uint_as_float(r[4 * i]) : 0.f;
              o[4 * i + 1] = a.y > 0.f ? __uint_as_float(r[4 * i + 1]) : 0.f;
              o[4 * i + 2] = a.z > 0.f ? __uint_as_float(r[4 * i + 2]) : 0.f;
              o[4 * i + 3] = a.w > 0.f ? __uint_as_float(r[4 * i + 3]) : 0.f;
            }
          } else {
            const uint4* a4 = reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(p.act) + at);
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
          }
          store_row32<TF32>(p.C, at, o);
          if (p.dbias != nullptr) {
            // column sums over this warp's 32 rows, through a padded 32 x 33 transpose in the (now idle)
            // stage memory; lane i ends up with column i
            float* tile = staging + (warp - 2) * (32 * 33);
            __syncwarp();
#pragma unroll
            for (int i = 0; i < 32; ++i) tile[lane * 33 + i] = o[i];
            __syncwarp();
            float cs = 0.f;
#pragma unroll
            for (int r = 0; r < 32; ++r) cs += tile[r * 33 + lane];
            colsum[(mt * 4 + q) * BN + c * 32 + lane] = cs;
          }
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
            if (!TF32 && p.Wb != nullptr) {
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
    if (EPI == EPI_FWD && p.head.W != nullptr) {
      // ---- the output layer, finished by the last CTA of the replica ---------------------------------
      const TcHead& hd = p.head;
      const int parts = gridDim.x;                 // CTAs that hold columns of this replica's rows
      const int tid = q * 32 + lane;               // this thread's row inside a row block (its TMEM lane)
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        float4* dst = reinterpret_cast<float4*>(hd.part + (((int64_t)g * parts + blockIdx.x) * p.M + mt * BM + tid) * kHeadMax);
#pragma unroll
        for (int i = 0; i < kHeadMax / 4; ++i)
          dst[i] = make_float4(hl[mt][4 * i], hl[mt][4 * i + 1], hl[mt][4 * i + 2], hl[mt][4 * i + 3]);
      }
      __threadfence();
      asm volatile("bar.sync 1, 128;" ::: "memory");
      uint32_t* flag = reinterpret_cast<uint32_t*>(smem + (SPLIT > 1 ? BN * BM * 4 : 0));   // idle stage memory
      if (tid == 0) *flag = (atomicInc(hd.counters + g, (unsigned)parts - 1) == (unsigned)parts - 1) ? 1u : 0u;
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (*flag != 0u) {
        __threadfence();
        const float invB = 1.0f / (float)p.M;
        float lsum = 0.f;
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          const int b = mt * BM + tid;
          float z[kHeadMax];
#pragma unroll
          for (int cls = 0; cls < kHeadMax; ++cls)
            z[cls] = (hd.bias != nullptr && cls < hd.C) ? hd.bias[(int64_t)g * hd.w_gstride + cls] : 0.f;
          for (int pt = 0; pt < parts; ++pt) {          // fixed order: column block by column block
            const float4* src = reinterpret_cast<const float4*>(hd.part + (((int64_t)g * parts + pt) * p.M + b) * kHeadMax);
#pragma unroll
            for (int i = 0; i < kHeadMax / 4; ++i) {
              const float4 v = __ldcg(src + i);
              z[4 * i] += v.x; z[4 * i + 1] += v.y; z[4 * i + 2] += v.z; z[4 * i + 3] += v.w;
            }
          }
          float loss;
          float d[kHeadMax];
          if (hd.kind == LS_LOSS_SOFTMAX_CE) {
            const int label = h_label[mt];
            float mx = z[0];
#pragma unroll
            for (int cls = 1; cls < kHeadMax; ++cls) if (cls < hd.C) mx = fmaxf(mx, z[cls]);
            float sum = 0.f, zy = mx;
#pragma unroll
            for (int cls = 0; cls < kHeadMax; ++cls)
              if (cls < hd.C) {
                d[cls] = expf(z[cls] - mx);
                sum += d[cls];
                if (cls == label) zy = z[cls];
              }
            loss = (mx + logf(sum)) - zy;
#pragma unroll
            for (int cls = 0; cls < kHeadMax; ++cls)
              if (cls < hd.C) d[cls] = (d[cls] / sum - (cls == label ? 1.f : 0.f)) * invB;
          } else {
            const float res = z[0] - h_target[mt];
            loss = 0.5f * res * res;
            d[0] = res * invB;
          }
          hd.row_loss[(int64_t)g * p.M + b] = loss;
          lsum += loss;
          if (hd.dZ != nullptr) {
#pragma unroll
            for (int cls = 0; cls < kHeadMax; ++cls)
              if (cls < hd.C) hd.dZ[((int64_t)g * p.M + b) * hd.C + cls] = d[cls];
          }
        }
        if (!hd.defer_loss && hd.loss_out != nullptr) {
          // mean of the row losses: lanes, then the four warps in order
#pragma unroll
          for (int o2 = 16; o2 > 0; o2 >>= 1) lsum += __shfl_xor_sync(0xffffffffu, lsum, o2);
          float* wsum = reinterpret_cast<float*>(flag) + 8;
          if (lane == 0) wsum[q] = lsum;
          asm volatile("bar.sync 1, 128;" ::: "memory");
          if (tid == 0) hd.loss_out[g] = (wsum[0] + wsum[1] + wsum[2] + wsum[3]) * invB;
        }
      }
    }
    if (EPI == EPI_DX && p.dbias != nullptr) {
      // all four epilogue warps (and only they) meet here; then one thread per column adds the partial
      // sums in a fixed order and applies v <- mu v + g, b <- b - eta v
      asm volatile("bar.sync 1, 128;" ::: "memory");
      for (int t = threadIdx.x - 64; t < CPR; t += 128) {
        float gsum = 0.f;
#pragma unroll
        for (int i = 0; i < MT * 4; ++i) gsum += colsum[i * BN + t];
        const int64_t at = (int64_t)g * p.dbias_gstride + n0 + rank * CPR + t;
        float step = gsum;
        if (p.mu != 0.f) {
          step = fmaf(p.mu, p.dvbias[at], gsum);
          p.dvbias[at] = step;
        }
        p.dbias[at] = fmaf(-p.lr, step, p.dbias[at]);
      }
    }
    tc_fence_before_sync();
  }
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// ---- bf16 forward / backward on CTA pairs ----------------------------------------------------------
// A 256 x 512 output tile per cluster of two CTAs (cta_group::2).  Every tcgen05.mma spans both SMs: a CTA
// supplies its 128 rows of A and its half (128 of 256 columns) of each of the two B blocks, and keeps its 128
// rows x 512 columns of the product in its own tensor memory.  Per stage a CTA brings in 48 KB (16 KB of A,
// 32 KB of B) for 128 x 512 x 64 products, against 64 KB for the same work on one CTA, and the tensor core
// reads each B element from shared memory once per pair instead of once per row block.
//   warp 0   TMA producer (each CTA loads its own parts; completion is counted on the leader's barrier);
//            backward: as the stages are used for the last time it also brings this CTA's 128 x 512 block of
//            the layer's activations (the ReLU mask) into them
//   warp 1   leader CTA: issues the MMAs; commits arrive on the barriers of both CTAs
//   warps 2-5 epilogue of this CTA's 128 rows: bias + ReLU (forward) or mask (backward) on the accumulator,
//            outputs packed to bf16 into the (now idle) stage memory in the layout of a TMA box, and written
//            with bulk tensor stores of 64 rows x 128 bytes.  (With one st.global per thread and row the
//            epilogue took as long as half the main loop: 16-32 k cycles against 4-5 k now.)
constexpr int kPairStages = 4;
constexpr int kPairN = 512;          // columns of the pair's tile: two MMA blocks of 256
constexpr int kPairGroups = kPairN / 64;      // 64-column groups of the epilogue (one 128-byte box row each)
constexpr int kThreadsPair = 320;    // warp 0 producer, warp 1 MMA issuer, warps 2-9 epilogue (two per TMEM lane quarter)
struct SmemPair {
  static constexpr int kABytes = BM * KB_BYTES;                 // this CTA's 128 rows
  static constexpr int kBBlockBytes = 128 * KB_BYTES;           // this CTA's half of one 256-column block
  static constexpr int kStageBytes = kABytes + 2 * kBBlockBytes;
  static constexpr int kRingBytes = kPairStages * kStageBytes;
  static constexpr int kBoxBytes = 64 * KB_BYTES;               // epilogue: 64 rows x 64 bf16
  static constexpr int kOutBytes = 2 * kPairGroups * kBoxBytes; // the CTA's 128 x 512 outputs (and mask) as boxes
  static constexpr int kColsumBytes = 2 * kPairN * 4;           // backward: column sums of the CTA's two row halves
  static constexpr int kBars = 2 * kPairStages + 1 + 2 * kPairGroups;
  static constexpr int kBarBytes = (kBars * 8 + 16 + 15) / 16 * 16;
  static constexpr int kBiasBytes = kPairN * 4;                 // forward: the bias of the tile's columns
  static constexpr int kTotal = 1024 + kRingBytes + kBarBytes + kBiasBytes;
  static_assert(kBarBytes % 16 == 0, "bias block alignment");
  static_assert(kOutBytes + kColsumBytes <= kRingBytes, "epilogue scratch");
  static_assert(kStageBytes % kBoxBytes == 0, "whole boxes per stage");
  static_assert(kTotal <= 227 * 1024, "shared memory budget");
};

__device__ __forceinline__ void tma_store_2d(const CUtensorMap* m, const void* src, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(
                   reinterpret_cast<uint64_t>(m)),
               "r"(smem_u32(src)), "r"(x), "r"(y)
               : "memory");
}

// tmC: the output [groups*M][N] as boxes of 64 rows x 64 bf16 (128-byte swizzle); tmMask (backward): the
// activations of the layer, same shape and boxes.
template <bool B_MN, int EPI>
__global__ void __launch_bounds__(kThreadsPair, 1)
tc_gemm_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const __grid_constant__ CUtensorMap tmC, const __grid_constant__ CUtensorMap tmMask, const Params p) {
  using L = SmemPair;
  constexpr int ELEMS = 64, MMA_K = 16, STAGES = kPairStages;
  constexpr int CHUNK_BYTES = ELEMS * KB_BYTES;
  constexpr uint32_t IDESC = make_idesc(1u, false, B_MN, 256, 256);
  constexpr uint32_t TMEM_COLS = kPairN;
  static_assert(EPI == EPI_FWD || EPI == EPI_DX, "forward / backward only");

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* stage_base = smem;
  float* colsum = reinterpret_cast<float*>(smem + L::kOutBytes);            // [2][kPairN]
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + L::kRingBytes);
  uint64_t* empty = full + STAGES;
  uint64_t* acc_full = empty + STAGES;
  uint64_t* mask_full = acc_full + 1;                           // [kPairGroups]
  uint64_t* box_done = mask_full + kPairGroups;                 // [kPairGroups] both row halves of a group written
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(box_done + kPairGroups);
  int* next_box = reinterpret_cast<int*>(tmem_slot + 1);        // backward: boxes whose column sums have been taken
  float* bias_s = reinterpret_cast<float*>(smem + L::kRingBytes + L::kBarBytes);   // [kPairN]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)cluster_ctarank();                    // 0: leader
  const int g = blockIdx.z;
  const int m0 = blockIdx.y * 256 + rank * BM;                // first row of this CTA inside the replica
  const int n0 = (int)(blockIdx.x >> 1) * kPairN;             // first column of the pair
  const int num_kb = p.K / ELEMS;
  const int out_row0 = g * p.M + m0;                          // first row of this CTA in the output / mask tensor

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(acc_full, 1);
    for (int i = 0; i < kPairGroups; ++i) { mbar_init(&mask_full[i], 1); mbar_init(&box_done[i], 2); }
    *next_box = 0;
    fence_mbar_init();
    prefetch_tmap(&tmA);
    prefetch_tmap(&tmB);
    prefetch_tmap(&tmC);
    if (EPI == EPI_DX) prefetch_tmap(&tmMask);
  }
  if (warp == 1) {
    tmem_alloc_pair(tmem_slot, TMEM_COLS);
    tmem_relinquish_pair();
  }
  tc_fence_before_sync();
  cluster_sync_all();       // both CTAs' barriers exist before either signals the other
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  grid_dep_wait();
  grid_dep_launch();

  float dx_pb = 0.f, dx_pvb = 0.f;      // backward: the bias / momentum element this thread updates
  if (warp == 0) {
    if (elect_one()) {
      const uint64_t pol_a = l2_policy(2), pol_b = l2_policy(1);
      const int a_base = operand_row_base(p.a, g);
      const int zb = p.b.z0 + g * p.b.z_step;
      const bool b_panel = p.b.rank3 == 2;
      const uint32_t full_leader = map_to_rank(smem_u32(&full[0]), 0);
      bool ok = true;
      for (int kb = 0; kb < num_kb; ++kb) {
        const int s = kb % STAGES;
        if (kb >= STAGES && !mbar_wait(&empty[s], ((kb / STAGES) - 1) & 1)) { atomicExch(p.err_flag, 21); ok = false; break; }
        if (rank == 0) mbar_expect_tx(&full[s], 2 * L::kStageBytes);      // both CTAs' bytes
        const uint32_t bar = full_leader + (uint32_t)(s * 8);
        uint8_t* sa = stage_base + s * L::kStageBytes;
        uint8_t* sb = sa + L::kABytes;
        const int k0 = kb * ELEMS;
#pragma unroll
        for (int c = 0; c < 2; ++c)
          tma_load_2d_pair(sa + c * CHUNK_BYTES, &tmA, bar, k0, a_base + m0 + c * 64, pol_a);
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          const int nb = n0 + j * 256 + rank * 128;       // this CTA's 128 columns of block j
#pragma unroll
          for (int c = 0; c < 2; ++c) {
            uint8_t* d = sb + j * L::kBBlockBytes + c * CHUNK_BYTES;
            const int x = B_MN ? nb + c * 64 : k0, y = B_MN ? k0 : nb + c * 64;
            if (b_panel) tma_load_4d_pair(d, &tmB, bar, 0, y, x >> 6, zb, pol_b);    // x is a multiple of 64
            else tma_load_3d_pair(d, &tmB, bar, x, y, zb, pol_b);
          }
        }
      }
      if (EPI == EPI_DX && ok) {
        // the mask: box b = (column group b / 2, row half b % 2) goes to bytes [b, b + 1) * 8 KB of the ring;
        // a stage is overwritten once the MMAs of its last use have completed
        for (int i = 0; i < kPairGroups; ++i) mbar_expect_tx(&mask_full[i], 2 * L::kBoxBytes);
        constexpr int kBoxesPerStage = L::kStageBytes / L::kBoxBytes;
        for (int i = 0; i < STAGES && ok; ++i) {
          const int s = (num_kb + i) % STAGES;                       // in the order of their last use
          const int uses = (num_kb - s + STAGES - 1) / STAGES;
          if (uses > 0 && !mbar_wait(&empty[s], (uses - 1) & 1)) { atomicExch(p.err_flag, 24); ok = false; break; }
          for (int b = s * kBoxesPerStage; b < (s + 1) * kBoxesPerStage && b < 2 * kPairGroups; ++b)
            tma_load_2d(smem + b * L::kBoxBytes, &tmMask, &mask_full[b >> 1], n0 + (b >> 1) * 64,
                        out_row0 + (b & 1) * 64);
        }
      }
    }
  } else if (warp == 1) {
    if (rank == 0 && elect_one()) {
      bool ok = true;
      for (int kb = 0; kb < num_kb; ++kb) {
        const int s = kb % STAGES;
        if (!mbar_wait(&full[s], (kb / STAGES) & 1)) { atomicExch(p.err_flag, 22); ok = false; break; }
        tc_fence_after_sync();
        const uint32_t a_addr = smem_u32(stage_base + s * L::kStageBytes);
        const uint32_t b_addr = a_addr + L::kABytes;
#pragma unroll
        for (int k = 0; k < ELEMS / MMA_K; ++k) {
          const uint32_t b_adv = B_MN ? k * MMA_K * KB_BYTES : k * 32;
          const uint32_t b_lbo = B_MN ? CHUNK_BYTES : 16;
          const uint64_t da = make_smem_desc(a_addr + k * 32, 16, 1024, kSwizzle128B);
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            const uint64_t db = make_smem_desc(b_addr + j * L::kBBlockBytes + b_adv, b_lbo, 1024, kSwizzle128B);
            mma_bf16_pair(tmem_base + (uint32_t)(j * 256), da, db, IDESC, (kb | k) != 0 ? 1u : 0u);
          }
        }
        mma_commit_pair(&empty[s]);
      }
      if (ok) mma_commit_pair(acc_full);
    }
  } else {
    // ---- epilogue of this CTA's 128 rows x 512 columns: warps 2-5 take columns 0..255, warps 6-9 the rest ----
    const int q = warp & 3;                  // TMEM lanes 32 q .. 32 q + 31
    const int cs = (warp - 2) >> 2;          // column half of the tile
    const int half = q >> 1;                 // rows 64 half .. of the CTA: one TMA box with the other warp of the half
    const int rih = (q & 1) * 32 + lane;     // this thread's row inside the box
    const int et = (int)threadIdx.x - 64;    // 0..255 among the epilogue threads
    const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
    // while the products run: the bias of the tile's columns goes to shared memory (forward), and the bias
    // elements that this thread will update are requested (backward)
    if (EPI == EPI_FWD) {
      if (et < kPairN / 4) {
        float4 bv = make_float4(0.f, 0.f, 0.f, 0.f);
        if (p.bias) bv = __ldg(reinterpret_cast<const float4*>(p.bias + (int64_t)g * p.bias_gstride + n0) + et);
        reinterpret_cast<float4*>(bias_s)[et] = bv;
      }
      asm volatile("bar.sync 1, 256;" ::: "memory");
    } else if (p.dbias != nullptr) {
      const int64_t at = (int64_t)g * p.dbias_gstride + n0 + rank * 256 + et;
      dx_pb = p.dbias[at];
      if (p.mu != 0.f) dx_pvb = p.dvbias[at];
    }
    bool ok = mbar_wait(acc_full, 0);
    ok = __all_sync(0xffffffffu, ok);
    tc_fence_after_sync();
    if (!ok && lane == 0) atomicExch(p.err_flag, 23);
    if (ok) {
      // the accumulator is read one 32-column block ahead of the arithmetic
      constexpr int kBlocks = kPairN / 64;           // 32-column blocks per warp
      const int c_begin = cs * kBlocks;
      uint32_t r[2][32];
      tmem_ld_32x32(taddr + c_begin * 32, r[0]);
#pragma unroll
      for (int ci = 0; ci < kBlocks; ++ci) {
        const int c = c_begin + ci;
        const int grp = c >> 1, sub = c & 1;
        uint8_t* box = smem + (grp * 2 + half) * L::kBoxBytes;
        uint8_t* myrow = box + rih * 128;
        tmem_ld_wait();
        if (ci + 1 < kBlocks) tmem_ld_32x32(taddr + (c + 1) * 32, r[(ci + 1) & 1]);
        if (EPI == EPI_DX && sub == 0 && ok) {
          // (after a failed wait the loop goes on without the mask, so that every barrier below is still met)
          ok = __all_sync(0xffffffffu, mbar_wait(&mask_full[grp], 0));
          if (!ok && lane == 0) atomicExch(p.err_flag, 25);
        }
        float o[32];
        if (EPI == EPI_FWD) {
          const float4* bias4 = reinterpret_cast<const float4*>(bias_s + c * 32);
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float4 bv = bias4[i];
            const float b4[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float v = __uint_as_float(r[ci & 1][4 * i + e]) + b4[e];
              o[4 * i + e] = (p.relu && !(v > 0.f)) ? 0.f : v;
            }
          }
        } else {
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const uint4 u = *reinterpret_cast<const uint4*>(myrow + (((sub * 4 + i) ^ (rih & 7)) << 4));
            const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              // a bf16 is positive iff it is non-zero with the sign bit clear
              const uint32_t lo = w[j] & 0xFFFFu, hi = w[j] >> 16;
              o[i * 8 + j * 2] = (lo != 0 && lo < 0x8000u) ? __uint_as_float(r[ci & 1][i * 8 + j * 2]) : 0.f;
              o[i * 8 + j * 2 + 1] = (hi != 0 && hi < 0x8000u) ? __uint_as_float(r[ci & 1][i * 8 + j * 2 + 1]) : 0.f;
            }
          }
        }
        // 32 outputs = four 16-byte pieces of this thread's box row (pieces are XOR-swizzled by the row)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          uint32_t u[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            __nv_bfloat162 t = __floats2bfloat162_rn(o[8 * i + 2 * e], o[8 * i + 2 * e + 1]);
            u[e] = *reinterpret_cast<uint32_t*>(&t);
          }
          *reinterpret_cast<uint4*>(myrow + (((sub * 4 + i) ^ (rih & 7)) << 4)) = make_uint4(u[0], u[1], u[2], u[3]);
        }
        if (sub == 1) {
          // both warps of the half have written the box: hand it to the bulk-copy engine
          fence_proxy_async_smem();
          asm volatile("bar.sync %0, 64;" ::"r"(2 + half + 2 * cs) : "memory");
          if ((q & 1) == 0 && lane == 0) {
            tma_store_2d(&tmC, box, n0 + grp * 64, out_row0 + half * 64);
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            if (EPI == EPI_DX) mbar_arrive(&box_done[grp]);
          }
        }
      }
    }
    if ((q & 1) == 0 && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    tc_fence_before_sync();
  }
  if (EPI == EPI_DX && p.dbias != nullptr) {
    // Column sums of the tile for the bias update of the layer below (the values as stored, i.e. rounded to bf16,
    // like the stand-alone bias kernel).  A box is 64 rows x 64 columns; whichever warp is free takes the next one
    // (producer and MMA warps at once, the epilogue warps as they finish), in the order in which the two sets of
    // epilogue warps complete them; lane cp adds columns 2 cp, 2 cp + 1 of the box in row order.
    __syncwarp();
    const int cp = lane;
    for (;;) {
      int k = 0;
      if (lane == 0) k = atomicAdd(next_box, 1);
      k = __shfl_sync(0xffffffffu, k, 0);
      if (k >= 2 * kPairGroups) break;
      const int grp = ((k >> 1) & 1) * (kPairGroups / 2) + (k >> 2), h = k & 1;
      if (!__all_sync(0xffffffffu, mbar_wait(&box_done[grp], 0))) break;     // (the epilogue has reported the failure)
      const uint8_t* box = smem + (grp * 2 + h) * L::kBoxBytes;
      float s0 = 0.f, s1 = 0.f;
#pragma unroll 8
      for (int r = 0; r < 64; ++r) {
        const uint32_t u = *reinterpret_cast<const uint32_t*>(box + r * 128 + (((cp >> 2) ^ (r & 7)) << 4) + (cp & 3) * 4);
        s0 += __uint_as_float(u << 16);
        s1 += __uint_as_float(u & 0xFFFF0000u);
      }
      colsum[h * kPairN + grp * 64 + 2 * cp] = s0;
      colsum[h * kPairN + grp * 64 + 2 * cp + 1] = s1;
    }
  }
  if (EPI == EPI_DX && p.dbias != nullptr) {
    // bias update of the layer below: column sums over the pair's 256 rows, added in row order (leader's
    // two halves, then the peer's) by the CTA that owns the column half
    cluster_sync_all();
    if (warp >= 2) {
      const uint32_t mine = smem_u32(colsum);
      const uint32_t src0 = map_to_rank(mine, 0), src1 = map_to_rank(mine, 1);
      {
        const int t = rank * 256 + (int)threadIdx.x - 64;
        float gsum = 0.f;
#pragma unroll
        for (int i = 0; i < 2; ++i) gsum += ld_cluster_f32(src0 + (uint32_t)((i * kPairN + t) * 4));
#pragma unroll
        for (int i = 0; i < 2; ++i) gsum += ld_cluster_f32(src1 + (uint32_t)((i * kPairN + t) * 4));
        const int64_t at = (int64_t)g * p.dbias_gstride + n0 + t;
        float step = gsum;
        if (p.mu != 0.f) {
          step = fmaf(p.mu, dx_pvb, gsum);
          p.dvbias[at] = step;
        }
        p.dbias[at] = fmaf(-p.lr, step, dx_pb);
      }
    }
  }
  // neither CTA leaves (or frees tensor memory) while the other may still read its shared memory or
  // receive an arrival from it
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc_pair(tmem_base, TMEM_COLS);
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

template <bool TF32, int BN, bool A_MN, bool B_MN, int EPI, int STAGES, int SPLIT = 1, int MT = 1>
int launch_one(const TcOperandMaps& mp, const Params& p, int groups, cudaStream_t st) {
  using L = Smem<TF32, BN, STAGES, MT>;
  auto kern = tc_gemm_kernel<TF32, BN, A_MN, B_MN, EPI, STAGES, SPLIT, MT>;
  static uint64_t configured = 0;        // one bit per device
  {
    cudaError_t e = allow_dynamic_smem(kern, (int)(L::kTotal), &configured);
    if (e != cudaSuccess) return e;
  }
  dim3 grid((unsigned)(p.N / BN * SPLIT), (unsigned)(p.M / (BM * MT)), (unsigned)groups);
  return launch_dep(kern, grid, dim3(TF32 ? kThreadsFp32 : kThreadsBf16), L::kTotal, st, SPLIT, *mp.a, *mp.b, p);
}

template <bool B_MN, int EPI>
int launch_pair(const TcOperandMaps& mp, const CUtensorMap* c_map, const CUtensorMap* mask_map, const Params& p,
                int groups, cudaStream_t st) {
  auto kern = tc_gemm_pair_kernel<B_MN, EPI>;
  static uint64_t configured = 0;        // one bit per device
  {
    cudaError_t e = allow_dynamic_smem(kern, (int)(SmemPair::kTotal), &configured);
    if (e != cudaSuccess) return e;
  }
  dim3 grid((unsigned)(p.N / kPairN * 2), (unsigned)(p.M / 256), (unsigned)groups);
  return launch_dep(kern, grid, dim3(kThreadsPair), SmemPair::kTotal, st, 2, *mp.a, *mp.b, *c_map,
                    mask_map ? *mask_map : *c_map, p);
}
// bf16 shapes that the pair kernel covers
bool pair_shape_ok(int M, int N, int K) { return M % 256 == 0 && N % kPairN == 0 && K % 64 == 0; }

// fp32 forward / backward: tile width and K split.  128-wide tiles when N allows; K is split over a
// cluster while that keeps the grid within one wave of SMs and every slice keeps whole stages.
template <bool A_MN, bool B_MN, int EPI>
int launch_fp32(const TcOperandMaps& mp, const Params& p, int groups, cudaStream_t st) {
  const int bn = (p.N % 128 == 0) ? 128 : 64;
  const int tiles = (p.M / BM) * (p.N / bn) * groups;
  const int num_kb = p.K / 32;
  int split = 1;
  const int max_split = bn == 128 ? 4 : 2;      // every CTA of the cluster finishes at least 32 columns
  while (split < max_split && tiles * split * 2 <= 148 && num_kb % (split * 2) == 0 && num_kb / (split * 2) >= 4)
    split *= 2;
  if (bn == 128) {
    if (split == 4) return launch_one<true, 128, A_MN, B_MN, EPI, 4, 4>(mp, p, groups, st);
    if (split == 2) return launch_one<true, 128, A_MN, B_MN, EPI, 4, 2>(mp, p, groups, st);
    return launch_one<true, 128, A_MN, B_MN, EPI, 4, 1>(mp, p, groups, st);
  }
  if (split == 2) return launch_one<true, 64, A_MN, B_MN, EPI, 4, 2>(mp, p, groups, st);
  return launch_one<true, 64, A_MN, B_MN, EPI, 4, 1>(mp, p, groups, st);
}

int make_map(CUtensorMap* out, const void* base, bool fp32, bool mn32, bool block32, int rank, int64_t rows,
             int64_t cols, int64_t groups, int64_t gstride, int box_rows = 0) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return cudaErrorNotSupported;
  const cuuint64_t eb = fp32 ? 4 : 2;
  const cuuint32_t elems = (cuuint32_t)(KB_BYTES / eb);
  cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)groups};
  cuuint64_t strides[2] = {(cuuint64_t)cols * eb, (cuuint64_t)gstride * eb};
  // K-major reads take boxes of 64 rows; MN-major reads (and the 32 x 32 blocks of the update kernel) of
  // fp32 tensors take 32 rows.  For bf16 both are 64.
  cuuint32_t box[3] = {elems, (fp32 && !mn32 && !block32) ? 64u : elems, 1};
  if (box_rows > 0) box[1] = (cuuint32_t)box_rows;
  cuuint32_t es[3] = {1, 1, 1};
  CUresult r = fn(out, fp32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank,
                  const_cast<void*>(base), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  (fp32 && mn32) ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_128B,
                  block32 ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B : CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

}  // namespace

// 2-D map over a row-major matrix [rows][cols] of bf16 or fp32; box = 128 bytes x (64 | 32) rows, 128-byte
// swizzle.  mn32: the fp32 tensor will be read as an MN-major operand (swizzle in 32-byte units).
int tc_make_map_2d(CUtensorMap* out, const void* base, bool fp32, bool mn32, int64_t rows, int64_t cols) {
  return make_map(out, base, fp32, mn32, false, 2, rows, cols, 1, 0);
}
// The same with boxes of box_rows rows (operand stages of the update kernel).
int tc_make_map_2d_rows(CUtensorMap* out, const void* base, bool fp32, bool mn32, int64_t rows, int64_t cols,
                        int box_rows) {
  return make_map(out, base, fp32, mn32, false, 2, rows, cols, 1, 0, box_rows);
}
// 3-D map over `groups` row-major matrices [rows][cols] that start every gstride elements.
int tc_make_map_3d(CUtensorMap* out, const void* base, bool fp32, bool mn32, int64_t rows, int64_t cols,
                   int64_t groups, int64_t gstride) {
  return make_map(out, base, fp32, mn32, false, 3, rows, cols, groups, gstride);
}
// 3-D map over fp32 matrices read and written in 32 x 32 blocks (128-byte swizzle, 16-byte units).
// blocked: the matrix is stored as 32 x 32 blocks (TileMap): block b is rows [32 b, 32 b + 32) of a
// [rows * cols / 32][32] matrix, i.e. box coordinates (0, 32 b).
int tc_make_block_map_3d(CUtensorMap* out, const void* base, int64_t rows, int64_t cols, int64_t groups,
                         int64_t gstride, bool blocked) {
  if (blocked) return make_map(out, base, true, false, true, 3, rows * cols / 32, 32, groups, gstride);
  return make_map(out, base, true, false, true, 3, rows, cols, groups, gstride);
}
int tc_make_panel_map(CUtensorMap* out, const void* base, int64_t rows, int64_t cols, int64_t groups, int64_t gstride) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return cudaErrorNotSupported;
  if (rows < 1 || cols < 64 || cols % 64 != 0 || groups < 1 || gstride < rows * cols || gstride % 8 != 0)
    return cudaErrorInvalidValue;
  cuuint64_t dims[4] = {64, (cuuint64_t)rows, (cuuint64_t)(cols / 64), (cuuint64_t)groups};
  cuuint64_t strides[3] = {128, (cuuint64_t)rows * 128, (cuuint64_t)gstride * 2};
  cuuint32_t box[4] = {64, 64, 1, 1};
  cuuint32_t es[4] = {1, 1, 1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, es,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

// The forward kernel can also evaluate a narrow output layer that follows when one CTA holds every row of
// its columns and the layer fits kHeadMax outputs.  Used for one row block (M = 128): with the 256-row
// bf16 tile the four epilogue warps carry two rows each and the separate output-layer kernel, which
// spreads the rows over the whole GPU, measured faster.
bool tc_fwd_fuses_head(bool fp32, int M, int N, int C) {
  (void)fp32;
  if (C < 1 || C > kHeadMax || N % 4 != 0) return false;
  return M == BM;
}
// upper bound of the CTAs that share a replica's rows (column blocks of at least 32 columns)
int tc_fwd_head_parts(int N) { return N / 32; }

// The backward kernel can finish the bias update when one CTA holds every row of its columns: M is one
// row block, or two with the 256-row bf16 tile.
bool tc_dx_fuses_bias(bool fp32, int M, int N) {
  if (M == BM) return true;
  return !fp32 && M == 2 * BM && N % 256 == 0;
}

// M output rows, N output columns, K contraction length of one group.
bool tc_shape_ok(bool fp32, int M, int N, int K) {
  if (M <= 0 || N <= 0 || K <= 0 || M % BM != 0) return false;
  return fp32 ? (N % 64 == 0 && K % 32 == 0) : (N % 128 == 0 && K % 64 == 0);
}

int launch_tc_fwd(const TcFwdArgs& a, cudaStream_t st, int64_t* launches) {
  Params p{};
  p.a = Operand{a.row_off, a.M, 0, 0, 0};
  p.b = Operand{nullptr, 0, a.w_z0, a.w_zstep, a.w_panel ? 2 : 1};
  p.M = a.M; p.N = a.N; p.K = a.K;
  p.bias = a.bias; p.bias_gstride = a.bias_gstride; p.relu = a.relu;
  p.C = a.C; p.err_flag = a.err_flag;
  p.head = a.head;
  if (p.head.W != nullptr && !tc_fwd_fuses_head(a.fp32, a.M, a.N, p.head.C)) return cudaErrorInvalidValue;
  if (launches) ++*launches;
  if (a.fp32) return launch_fp32<false, false, EPI_FWD>(a.maps, p, a.groups, st);
  if (a.allow_pair && p.head.W == nullptr && a.c_map != nullptr && pair_shape_ok(a.M, a.N, a.K))
    return launch_pair<false, EPI_FWD>(a.maps, a.c_map, nullptr, p, a.groups, st);
  if (a.N % 256 == 0 && a.M % 256 == 0) return launch_one<false, 256, false, false, EPI_FWD, 3, 1, 2>(a.maps, p, a.groups, st);
  if (a.N % 256 == 0) return launch_one<false, 256, false, false, EPI_FWD, 4>(a.maps, p, a.groups, st);
  return launch_one<false, 128, false, false, EPI_FWD, 4>(a.maps, p, a.groups, st);
}

int launch_tc_dx(const TcDxArgs& a, cudaStream_t st, int64_t* launches) {
  Params p{};
  p.a = Operand{nullptr, a.M, 0, 0, 0};
  p.b = Operand{nullptr, 0, 0, a.w_zstep, a.w_panel ? 2 : 1};
  p.M = a.M; p.N = a.N; p.K = a.K;
  p.C = a.C; p.act = a.act; p.err_flag = a.err_flag;
  if (a.bias != nullptr && tc_dx_fuses_bias(a.fp32, a.M, a.N)) {
    p.dbias = a.bias; p.dvbias = a.vbias; p.dbias_gstride = a.bias_gstride; p.lr = a.lr; p.mu = a.mu;
  }
  if (launches) ++*launches;
  if (a.fp32) return launch_fp32<false, true, EPI_DX>(a.maps, p, a.groups, st);
  if (a.allow_pair && a.c_map != nullptr && a.act_map != nullptr && pair_shape_ok(a.M, a.N, a.K))
    return launch_pair<true, EPI_DX>(a.maps, a.c_map, a.act_map, p, a.groups, st);
  if (a.N % 256 == 0 && a.M % 256 == 0) return launch_one<false, 256, false, true, EPI_DX, 3, 1, 2>(a.maps, p, a.groups, st);
  if (a.N % 256 == 0) return launch_one<false, 256, false, true, EPI_DX, 4>(a.maps, p, a.groups, st);
  return launch_one<false, 128, false, true, EPI_DX, 4>(a.maps, p, a.groups, st);
}

int launch_tc_dw(const TcDwArgs& a, cudaStream_t st, int64_t* launches) {
  Params p{};
  p.a = Operand{nullptr, a.B, 0, 0, 0};
  p.b = Operand{a.row_off, a.B, 0, 0, 0};
  p.M = a.M; p.N = a.N; p.K = a.B;
  p.W = a.W; p.V = a.V; p.Wb = a.Wb; p.w_gstride = a.w_gstride; p.lr = a.lr; p.mu = a.mu;
  p.err_flag = a.err_flag;
  if (launches) ++*launches;
  if (a.fp32) {
    if (a.N % 128 == 0) return launch_one<true, 128, true, true, EPI_DW, 4>(a.maps, p, a.groups, st);
    return launch_one<true, 64, true, true, EPI_DW, 4>(a.maps, p, a.groups, st);
  }
  return launch_one<false, 128, true, true, EPI_DW, 3>(a.maps, p, a.groups, st);
}

}  // namespace ls
