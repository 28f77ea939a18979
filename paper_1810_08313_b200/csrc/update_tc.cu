// Weight gradient + SGD-momentum update as one persistent, warp-specialised
// streaming kernel (Section 2 mini-batch SGD update; Section 5.3 momentum):
//
//     G = dZ^T A  (per replica, 128 x 128 tiles on tcgen05, accumulator in TMEM)
//     v <- mu v + G ;  W <- W - eta v ;  refresh the operand copy of W
//
// for every layer whose shapes fill tensor-core tiles, in ONE launch: the updates of different layers do
// not depend on one another, so their tiles form one list (largest layer first) that the CTAs walk.
// Every CTA takes the same number of whole 128 x 128 tiles; the tiles left over after those rounds are cut
// into column strips (32 columns for fp32, 64 for bf16) that are spread over all CTAs, so that the last
// round is a fraction of a tile long instead of a whole tile on a few SMs.
// The gradient never leaves the SM.  The kernel is bound by the read-modify-write
// of W and v (16 bytes per parameter with momentum, plus the bf16 copy of a bf16 model), so it
// is built as a stream: one CTA per SM walks over output tiles, and
//
//   warp 0      TMA producer of the dZ / A operand tiles (ring of stages)
//   warp 1      tcgen05.mma issuer; two TMEM accumulators, so the products of tile t+1
//               overlap the update of tile t
//   warps 2-3   fp32 models: write lo = x - tf32(x) of each operand stage beside it in shared
//               memory (three tf32 MMAs per product: lo*hi + hi*lo + hi*hi)
//   warps 4-7   update warps.  Each owns 32 rows of the tile and a private ring of
//               shared-memory slots: TMA loads bring its 32 x 32 blocks of W and v in
//               (issued up to a whole tile ahead), the warp adds the TMEM gradient in
//               place, and TMA stores write the blocks back.  Loads and stores are
//               asynchronous bulk copies, so tens of KB per SM are always in flight.
//
// Every mbarrier wait is bounded (see tc_ptx.cuh); a wait that runs out sets
// *err_flag and the CTA drains its copies, frees its tensor memory and returns.
#include "ls_internal.h"
#include "tc_ptx.cuh"

namespace ls {
namespace {

using namespace ptx;

constexpr int BM = 128, BN = 128;
constexpr int KB_BYTES = 128;
constexpr int kThreads = 256;
constexpr int kSlotBytes = 8192;       // one 32 x 32 fp32 block of W (4 KB) and of v (4 KB)

constexpr int kMaxLayers = 4;          // layers per launch
constexpr int kRowsFp32 = 16;          // mini-batch rows per operand stage: the TMA boxes of the operand maps
constexpr int kRowsBf16 = 64;          // are this many rows high (tc_update_box_rows)

struct ULayer {
  int N;                               // in features (row length of W)
  int n_tiles;                         // N / BN
  int tiles_per_group;                 // (M / BM) * (N / BN)
  int tile_begin;                      // first tile of this layer in the launch's list
  const int64_t* b_row_off;            // layer input = dataset rows: first row of replica g, else null
  __nv_bfloat16* Wb;                   // bf16 copy of W (bf16 models) or null
  int blocked;                         // W, v stored as 32 x 32 blocks (TileMap): box coordinates differ
  int pM;                              // rows of W when Wb is kept in 64-column panels (TileMap), else 0: row-major
};
struct UParams {
  ULayer layer[kMaxLayers];
  int n_layers, total_tiles;
  int full_rounds;                     // whole tiles per CTA; tile t of round n on CTA b is b + n * gridDim.x
  int tail_units;                      // column strips of the left-over tiles, strip u on CTA u % gridDim.x
  int K, groups;                       // batch, replicas
  int shared_state;                    // 1: all replicas enter with the same W, v: read the synchronized copy (maps.wl / vl,
                                       //    one vector) instead of each replica's own, and walk the list replica-minor
  int rows_per_group;                  // = batch
  float lr, mu;
  int64_t w_gstride;                   // elements between replicas
  int* err_flag;
};
// dZ_l (a), layer input (b), weights and momentum (w, v) of every layer of the launch
// (w, v: where the new values are stored; wl, vl: where the old ones are loaded from -- the same tensors, or the
// synchronized copy when every replica holds the same values)
struct alignas(64) UMaps {
  CUtensorMap a[kMaxLayers], b[kMaxLayers], w[kMaxLayers], v[kMaxLayers], wl[kMaxLayers], vl[kMaxLayers];
};

struct Tile { int layer, g, m0, n0; };
// A unit of work: 32-column blocks [c0, c0 + nc) of a tile (nc = 4: the whole tile).
struct Unit { Tile tl; int c0, nc; };
__device__ __forceinline__ Tile decode_tile(const UParams& p, int t) {
  int l = 0;
#pragma unroll
  for (int i = 1; i < kMaxLayers; ++i)
    if (i < p.n_layers && t >= p.layer[i].tile_begin) l = i;
  const int r = t - p.layer[l].tile_begin;
  const int tpg = p.layer[l].tiles_per_group, nt = p.layer[l].n_tiles;
  // replica-minor when the replicas share their old state: the CTAs that read one tile of it run side by side
  const int g = p.shared_state ? r % p.groups : r / tpg, rem = p.shared_state ? r / p.groups : r % tpg;
  return Tile{l, g, (rem / nt) * BM, (rem % nt) * BN};
}

// Operand stages are filled by TMA; fp32 models add one buffer for the lo parts of the stage in use.
// KS: K-rows (mini-batch rows) per stage.
template <bool TF32, int STAGES, int R, int KS>
struct USmem {
  static constexpr int kLoStages = TF32 ? 1 : 0;
  static constexpr int kStageBytes = (BM + BN) * KS * (TF32 ? 4 : 2);
  static constexpr int kOperandBytes = (STAGES + kLoStages) * kStageBytes;
  static constexpr int kRingBytes = 4 * R * kSlotBytes;
  static constexpr int kBars = 2 * STAGES + 2 + 4 + 4 * R;
  static constexpr int kTotal = 1024 + kOperandBytes + kRingBytes + kBars * 8 + 16;
  static_assert(kTotal <= 227 * 1024, "shared memory budget");
};

__device__ __forceinline__ void tma_store_3d(const CUtensorMap* m, const void* src, int x, int y, int z) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];" ::"l"(
                   reinterpret_cast<uint64_t>(m)),
               "r"(smem_u32(src)), "r"(x), "r"(y), "r"(z)
               : "memory");
}
// Box coordinates of the 32 x 32 block at row y, column x of a matrix with rows of ldw elements: (x, y) in a
// row-major matrix; in blocked storage block b is rows 32 b .. of a [.][32] matrix.
__device__ __forceinline__ void block_coords(int blocked, int ldw, int& x, int& y) {
  if (blocked) {
    y = ((y >> 5) * (ldw >> 5) + (x >> 5)) << 5;
    x = 0;
  }
}
// Where, inside a replica's bf16 copy of W, the piece of row `row` that starts at column `col` begins (a piece
// never crosses a multiple of 64 columns).
__device__ __forceinline__ int64_t copy_index(int pM, int ldw, int row, int col) {
  return pM ? ((int64_t)(col >> 6) * pM + row) * 64 + (col & 63) : (int64_t)row * ldw + col;
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// one 32-byte (whole sector) store; p must be 32-byte aligned
__device__ __forceinline__ void st_global_v8(void* p, const uint32_t (&v)[8]) {
  asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]),
               "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
               : "memory");
}

template <int MNC, int KS>
__device__ __forceinline__ void issue_mn_tile(void* dst, const CUtensorMap* tm, uint64_t* bar, int tile0, int extent,
                                              int row0, uint64_t pol) {
  // MN-major operand: boxes of 128 bytes (MNC MN-elements) x KS K-rows, one per chunk of MN
  for (int c = 0; c < extent / MNC; ++c)
    tma_load_2d_hint(static_cast<char*>(dst) + c * KS * KB_BYTES, tm, bar, tile0 + c * MNC, row0, pol);
}

// n-th unit of CTA `b`; SUB strips per left-over tile
template <int SUB>
__device__ __forceinline__ Unit decode_unit(const UParams& p, int n, int b, int grid) {
  if (n < p.full_rounds) return Unit{decode_tile(p, b + n * grid), 0, 4};
  const int u = b + (n - p.full_rounds) * grid;
  constexpr int NC = 4 / SUB;
  return Unit{decode_tile(p, p.full_rounds * grid + u / SUB), (u % SUB) * NC, NC};
}

template <bool TF32, int STAGES, int R, int KS>
__global__ void __launch_bounds__(kThreads, 1)
tc_update_kernel(const __grid_constant__ UMaps maps, const __grid_constant__ UParams p) {
  using L = USmem<TF32, STAGES, R, KS>;
  constexpr int EB = TF32 ? 4 : 2;
  constexpr int MNC = KB_BYTES / EB;            // MN elements per operand chunk (one 128-byte row)
  constexpr int MMA_K = 32 / EB;
  constexpr int CHUNK_BYTES = KS * KB_BYTES;
  static_assert(KS % MMA_K == 0 && KS % 8 == 0, "whole MMAs and swizzle periods per stage");
  constexpr uint32_t IDESC = make_idesc(TF32 ? 2u : 1u, true, true, BM, BN);
  constexpr int SUB = TF32 ? 4 : 2;             // column strips per left-over tile (one operand chunk each)
  constexpr int NCS = 4 / SUB;                  // 32-column blocks per strip
  constexpr uint32_t IDESC_STRIP = make_idesc(TF32 ? 2u : 1u, true, true, BM, BN / SUB);
  constexpr uint32_t SW = TF32 ? kSwizzle128B_32B : kSwizzle128B;
  constexpr uint32_t SBO = TF32 ? 512 : 1024;
  constexpr int kABytes = BM * KS * EB;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* stage_base = smem;
  uint8_t* lo_buf = smem + STAGES * L::kStageBytes;
  uint8_t* ring_base = smem + L::kOperandBytes;
  uint64_t* full = reinterpret_cast<uint64_t*>(ring_base + L::kRingBytes);
  uint64_t* empty = full + STAGES;
  uint64_t* tmem_full = empty + STAGES;       // [2]
  uint64_t* tmem_empty = tmem_full + 2;       // [2]
  uint64_t* wv_full = tmem_empty + 2;         // [4][R]
  uint64_t* lo_full = wv_full + 4 * R;        // fp32: lo parts of the current stage written ...
  uint64_t* lo_empty = lo_full + 1;           // ... and read by the tensor core
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(lo_empty + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_kb = p.K / KS;
  const int bx = blockIdx.x, grid = gridDim.x;
  const int my_strips = bx < p.tail_units ? (p.tail_units - 1 - bx) / grid + 1 : 0;
  const int my_units = p.full_rounds + my_strips;
  const bool has_v = p.mu != 0.f;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(lo_full, 2); mbar_init(lo_empty, 1);
    for (int b = 0; b < 2; ++b) { mbar_init(&tmem_full[b], 1); mbar_init(&tmem_empty[b], 4); }
    for (int i = 0; i < 4 * R; ++i) mbar_init(&wv_full[i], 1);
    fence_mbar_init();
    for (int l = 0; l < p.n_layers; ++l) {
      prefetch_tmap(&maps.a[l]); prefetch_tmap(&maps.b[l]); prefetch_tmap(&maps.w[l]); prefetch_tmap(&maps.v[l]);
      prefetch_tmap(&maps.wl[l]); prefetch_tmap(&maps.vl[l]);
    }
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, 2 * BN);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  grid_dep_wait();        // the prologue above overlapped the previous kernel
  grid_dep_launch();

  if (warp == 0) {
    // ---- operand producer ---------------------------------------------------------
    if (elect_one()) {
      int it = 0;
      bool ok = true;
      // dZ and the layer inputs are re-read by every CTA that shares a row or column of tiles, while the
      // W / v stream passes through L2 once: keep the operands (measured: 802 -> 782 us on the bf16 MLP)
      const uint64_t pol = l2_policy(2);
      for (int n = 0; n < my_units && ok; ++n) {
        const Unit un = decode_unit<SUB>(p, n, bx, grid);
        const Tile tl = un.tl;
        const int a_row = tl.g * p.rows_per_group;
        const int64_t* b_off = p.layer[tl.layer].b_row_off;
        const int b_row = b_off ? (int)b_off[tl.g] : a_row;
        const CUtensorMap* tmA = &maps.a[tl.layer];
        const CUtensorMap* tmB = &maps.b[tl.layer];
        for (int kb = 0; kb < num_kb; ++kb, ++it) {
          const int s = it % STAGES;
          if (!mbar_wait(&empty[s], ((it / STAGES) & 1) ^ 1)) { atomicExch(p.err_flag, 11); ok = false; break; }
          mbar_expect_tx(&full[s], kABytes + un.nc * 32 * KS * EB);
          uint8_t* sa = stage_base + s * L::kStageBytes;
          uint8_t* sb = sa + kABytes;
          issue_mn_tile<MNC, KS>(sa, tmA, &full[s], tl.m0, BM, a_row + kb * KS, pol);
          issue_mn_tile<MNC, KS>(sb, tmB, &full[s], tl.n0 + un.c0 * 32, un.nc * 32, b_row + kb * KS, pol);
        }
      }
    }
  } else if (TF32 && (warp == 2 || warp == 3)) {
    // ---- splitter warps: the lo copy has the layout of the tile it comes from ------------
    const int tid = threadIdx.x - 64;
    const int total_it = my_units * num_kb;
    for (int it = 0; it < total_it; ++it) {
      const int s = it % STAGES;
      bool got = mbar_wait(&full[s], (it / STAGES) & 1);
      if (got && it >= 1) got = mbar_wait(lo_empty, (it - 1) & 1);
      if (!__all_sync(0xffffffffu, got)) {
        if (lane == 0) atomicExch(p.err_flag, 16);
        break;
      }
      split_lo_smem(smem_u32(stage_base + s * L::kStageBytes), smem_u32(lo_buf), L::kStageBytes, tid, 64);
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(lo_full);
    }
  } else if (warp == 1) {
    // ---- MMA issuer -----------------------------------------------------------------
    if (elect_one()) {
      int it = 0;
      bool ok = true;
      for (int n = 0; n < my_units && ok; ++n) {
        const int buf = n & 1;
        const uint32_t idesc = n < p.full_rounds ? IDESC : IDESC_STRIP;     // a strip is BN / SUB columns wide
        if (!mbar_wait(&tmem_empty[buf], ((n >> 1) & 1) ^ 1)) { atomicExch(p.err_flag, 12); break; }
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
        for (int kb = 0; kb < num_kb; ++kb, ++it) {
          const int s = it % STAGES;
          if (!mbar_wait(&full[s], (it / STAGES) & 1)) { atomicExch(p.err_flag, 13); ok = false; break; }
          if (TF32 && !mbar_wait(lo_full, it & 1)) { atomicExch(p.err_flag, 17); ok = false; break; }
          tc_fence_after_sync();
          const uint32_t a_addr = smem_u32(stage_base + s * L::kStageBytes);
          const uint32_t b_addr = a_addr + kABytes;
#pragma unroll
          for (int k = 0; k < KS / MMA_K; ++k) {
            const uint32_t adv = k * MMA_K * KB_BYTES;      // next MMA_K K-rows
            const uint64_t da = make_smem_desc(a_addr + adv, CHUNK_BYTES, SBO, SW);
            const uint64_t db = make_smem_desc(b_addr + adv, CHUNK_BYTES, SBO, SW);
            const uint32_t acc = (kb | k) != 0 ? 1u : 0u;
            if (TF32) {
              const uint64_t dal = make_smem_desc(smem_u32(lo_buf) + adv, CHUNK_BYTES, SBO, SW);
              const uint64_t dbl = make_smem_desc(smem_u32(lo_buf) + kABytes + adv, CHUNK_BYTES, SBO, SW);
              mma_tf32(d_tmem, dal, db, idesc, acc);
              mma_tf32(d_tmem, da, dbl, idesc, 1u);
              mma_tf32(d_tmem, da, db, idesc, 1u);
            } else {
              mma_bf16(d_tmem, da, db, idesc, acc);
            }
          }
          mma_commit(&empty[s]);
          if (TF32) mma_commit(lo_empty);
        }
        if (ok) mma_commit(&tmem_full[buf]);
      }
    }
  } else if (warp >= 4) {
    // ---- update warps -----------------------------------------------------------------
    const int q = warp & 3;
    uint8_t* my_ring = ring_base + q * R * kSlotBytes;
    uint64_t* my_full = wv_full + q * R;
    const int full_chunks = p.full_rounds * 4;
    const int my_chunks = full_chunks + my_strips * NCS;

    // chunk j of this CTA: the 32 x 32 block of rows q*32.. and column block c of unit n, where whole
    // tiles contribute four chunks each and strips NCS
    auto load_chunk = [&](int j) {
      if (j >= my_chunks) return;
      const int n = j < full_chunks ? (j >> 2) : p.full_rounds + (j - full_chunks) / NCS;
      const Unit un = decode_unit<SUB>(p, n, bx, grid);
      const Tile tl = un.tl;
      const int c = j < full_chunks ? (j & 3) : un.c0 + (j - full_chunks) % NCS;
      int y = tl.m0 + q * 32, x = tl.n0 + c * 32;
      block_coords(p.layer[tl.layer].blocked, p.layer[tl.layer].N, x, y);
      uint8_t* slot = my_ring + (j % R) * kSlotBytes;
      mbar_expect_tx(&my_full[j % R], has_v ? kSlotBytes : kSlotBytes / 2);
      const int z = p.shared_state ? 0 : tl.g;
      tma_load_3d(slot, &maps.wl[tl.layer], &my_full[j % R], x, y, z);
      if (has_v) tma_load_3d(slot + kSlotBytes / 2, &maps.vl[tl.layer], &my_full[j % R], x, y, z);
    };
    if (lane == 0)
      for (int j = 0; j < R; ++j) load_chunk(j);

    const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
    bool ok = true;
    int j = 0;
    for (int n = 0; n < my_units && ok; ++n) {
      const Unit un = decode_unit<SUB>(p, n, bx, grid);
      const Tile tl = un.tl;
      const int g = tl.g, m0 = tl.m0, n0 = tl.n0;
      const int ldw = p.layer[tl.layer].N;
      __nv_bfloat16* Wb = p.layer[tl.layer].Wb;
      const int buf = n & 1;
      ok = __all_sync(0xffffffffu, mbar_wait(&tmem_full[buf], (n >> 1) & 1));
      if (!ok) { if (lane == 0) atomicExch(p.err_flag, 14); break; }
      tc_fence_after_sync();
#pragma unroll 1
      for (int ci = 0; ci < un.nc; ++ci, ++j) {
        const int c = un.c0 + ci;          // column block inside the tile; the accumulator starts at the strip
        uint8_t* slot = my_ring + (j % R) * kSlotBytes;
        uint32_t r[32];
        tmem_ld_32x32(taddr + buf * BN + ci * 32, r);
        ok = __all_sync(0xffffffffu, mbar_wait(&my_full[j % R], (j / R) & 1));
        tmem_ld_wait();
        if (ci == un.nc - 1) {
          // the accumulator has been read: hand the TMEM buffer back to the MMA warp
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&tmem_empty[buf]);
        }
        if (!ok) { if (lane == 0) atomicExch(p.err_flag, 15); break; }
        // this thread's row of the 32 x 32 block; 16-byte pieces are XOR-swizzled by the row (128-byte swizzle)
        const int64_t at = (int64_t)g * p.w_gstride + copy_index(p.layer[tl.layer].pM, ldw, m0 + q * 32 + lane, n0 + c * 32);
        uint32_t cp[8];
#pragma unroll
        for (int jj = 0; jj < 8; ++jj) {
          const int off = lane * 128 + ((jj ^ (lane & 7)) << 4);
          float4 w = *reinterpret_cast<float4*>(slot + off);
          float ws[4] = {w.x, w.y, w.z, w.w};
          float vs[4] = {0.f, 0.f, 0.f, 0.f};
          if (has_v) {
            const float4 v = *reinterpret_cast<float4*>(slot + kSlotBytes / 2 + off);
            vs[0] = v.x; vs[1] = v.y; vs[2] = v.z; vs[3] = v.w;
          }
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float gr = __uint_as_float(r[jj * 4 + e]);
            const float step = has_v ? fmaf(p.mu, vs[e], gr) : gr;
            vs[e] = step;
            ws[e] = fmaf(-p.lr, step, ws[e]);
          }
          *reinterpret_cast<float4*>(slot + off) = make_float4(ws[0], ws[1], ws[2], ws[3]);
          if (has_v) *reinterpret_cast<float4*>(slot + kSlotBytes / 2 + off) = make_float4(vs[0], vs[1], vs[2], vs[3]);
          // operand copy of the new weights, collected so that it leaves in whole 32-byte sectors
          if (!TF32 && Wb != nullptr) {
            __nv_bfloat162 lo = __floats2bfloat162_rn(ws[0], ws[1]);
            __nv_bfloat162 hi = __floats2bfloat162_rn(ws[2], ws[3]);
            cp[(jj & 3) * 2] = *reinterpret_cast<uint32_t*>(&lo);
            cp[(jj & 3) * 2 + 1] = *reinterpret_cast<uint32_t*>(&hi);
            if ((jj & 3) == 3) st_global_v8(Wb + at + (jj - 3) * 4, cp);
          }
        }
        // make the in-place update visible to the bulk-copy engine, then write the blocks back
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          int y = m0 + q * 32, x = n0 + c * 32;
          block_coords(p.layer[tl.layer].blocked, ldw, x, y);
          tma_store_3d(&maps.w[tl.layer], slot, x, y, g);
          if (has_v) tma_store_3d(&maps.v[tl.layer], slot + kSlotBytes / 2, x, y, g);
          bulk_commit();
          // the slot used one chunk ago is free once its store has read shared memory: refill it
          bulk_wait_read<1>();
          if (j >= 1) load_chunk(j - 1 + R);
        }
        __syncwarp();
      }
    }
    if (lane == 0) bulk_wait_all();
    tc_fence_before_sync();
  }
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, 2 * BN);
  }
}

// ---- bf16 models whose layers are multiples of 256 wide: the same stream on CTA pairs ---------------------------
// Two CTAs of a cluster share every tcgen05.mma (cta_group::2): the pair's unit is a 256 x 256 block of W, CTA r
// owns rows 128 r .. of it.  A CTA stages its own 128 columns of dZ and HALF of the unit's 256 columns of the layer
// input per 64-row stage, i.e. the same 32 KB as the one-CTA kernel, for twice the products: cycle traces of that
// kernel show its update warps waiting for the products (one 32 KB operand stage, four loads in sequence per
// tile), and shared memory has no room for a second stage beside the W / v ring.  Everything else (the per-warp
// W / v rings, the update arithmetic, the left-over strips) is as in tc_update_kernel.
//   full[s]        on the leader: both CTAs' operand bytes of a stage
//   empty[s], tmem_full[b]   in each CTA, signalled by the leader's multicast commits
//   tmem_empty[b]  on the leader: the 8 update warps of the pair have read accumulator b
constexpr int PN = 256;                 // columns of a pair's unit
struct PLayer {
  int N, n_tiles, tiles_per_group, tile_begin;
  const int64_t* b_row_off;
  __nv_bfloat16* Wb;
  int blocked;
  int pM;                               // as in ULayer
};
struct PParams {
  PLayer layer[kMaxLayers];
  int n_layers;
  int full_rounds;                     // whole units per pair; unit t of round n on pair b is b + n * pairs
  int tail_units;                      // 128-column strips of the left-over units, strip u on pair u % pairs
  int K, rows_per_group;
  int groups, shared_state;            // as in UParams
  float lr, mu;
  int64_t w_gstride;
  int* err_flag;
};
struct PUnit { int layer, g, m0, n0, nc; };      // columns [n0, n0 + 32 nc) of rows [m0, m0 + 256)

__device__ __forceinline__ PUnit decode_punit(const PParams& p, int n, int pb, int pairs) {
  int t, c0 = 0, nc = PN / 32;
  if (n < p.full_rounds) {
    t = pb + n * pairs;
  } else {
    const int u = pb + (n - p.full_rounds) * pairs;
    t = p.full_rounds * pairs + (u >> 1);
    nc = PN / 64;
    c0 = (u & 1) * nc;
  }
  int l = 0;
#pragma unroll
  for (int i = 1; i < kMaxLayers; ++i)
    if (i < p.n_layers && t >= p.layer[i].tile_begin) l = i;
  const int r = t - p.layer[l].tile_begin;
  const int tpg = p.layer[l].tiles_per_group, nt = p.layer[l].n_tiles;
  const int g = p.shared_state ? r % p.groups : r / tpg, rem = p.shared_state ? r / p.groups : r % tpg;
  return PUnit{l, g, (rem / nt) * 256, (rem % nt) * PN + c0 * 32, nc};
}

constexpr int kPairThreads = 384;      // producer, MMA issuer, two idle warps, eight update warps
template <int R, int KS>
__global__ void __launch_bounds__(kPairThreads, 1)
tc_update_pair_kernel(const __grid_constant__ UMaps maps, const __grid_constant__ PParams p) {
  using L = USmem<false, 1, R, KS>;
  constexpr int MMA_K = 16;
  constexpr int CHUNK_BYTES = KS * KB_BYTES;
  constexpr int kABytes = BM * KS * 2;               // this CTA's 128 columns of dZ, KS rows
  constexpr uint32_t IDESC_FULL = make_idesc(1u, true, true, 256, PN);
  constexpr uint32_t IDESC_STRIP = make_idesc(1u, true, true, 256, PN / 2);

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* stage = smem;
  uint8_t* ring_base = smem + L::kOperandBytes;
  uint64_t* full = reinterpret_cast<uint64_t*>(ring_base + L::kRingBytes);
  uint64_t* empty = full + 1;
  uint64_t* tmem_full = empty + 1;            // [2]
  uint64_t* tmem_empty = tmem_full + 2;       // [2]
  uint64_t* wv_full = tmem_empty + 2;         // [4][R]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(wv_full + 4 * R);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)cluster_ctarank();
  const int num_kb = p.K / KS;
  const int pb = blockIdx.x >> 1, pairs = gridDim.x >> 1;
  const int my_strips = pb < p.tail_units ? (p.tail_units - 1 - pb) / pairs + 1 : 0;
  const int my_units = p.full_rounds + my_strips;
  const bool has_v = p.mu != 0.f;

  if (threadIdx.x == 0) {
    mbar_init(full, 1); mbar_init(empty, 1);
    for (int b = 0; b < 2; ++b) { mbar_init(&tmem_full[b], 1); mbar_init(&tmem_empty[b], 16); }
    for (int i = 0; i < 4 * R; ++i) mbar_init(&wv_full[i], 1);
    fence_mbar_init();
    for (int l = 0; l < p.n_layers; ++l) {
      prefetch_tmap(&maps.a[l]); prefetch_tmap(&maps.b[l]); prefetch_tmap(&maps.w[l]); prefetch_tmap(&maps.v[l]);
      prefetch_tmap(&maps.wl[l]); prefetch_tmap(&maps.vl[l]);
    }
  }
  if (warp == 1) {
    tmem_alloc_pair(tmem_slot, 2 * PN);
    tmem_relinquish_pair();
  }
  tc_fence_before_sync();
  cluster_sync_all();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  grid_dep_wait();
  grid_dep_launch();

  if (warp == 0) {
    // ---- operand producer (each CTA loads its own parts; the leader's barrier counts both) -----------
    if (elect_one()) {
      const uint64_t pol = l2_policy(2);
      const uint32_t full_leader = map_to_rank(smem_u32(full), 0);
      int it = 0;
      bool ok = true;
      for (int n = 0; n < my_units && ok; ++n) {
        const PUnit un = decode_punit(p, n, pb, pairs);
        const int a_row = un.g * p.rows_per_group;
        const int64_t* b_off = p.layer[un.layer].b_row_off;
        const int b_row = b_off ? (int)b_off[un.g] : a_row;
        const CUtensorMap* tmA = &maps.a[un.layer];
        const CUtensorMap* tmB = &maps.b[un.layer];
        const int bcols = un.nc * 16;                          // this CTA's half of the unit's columns
        for (int kb = 0; kb < num_kb; ++kb, ++it) {
          if (!mbar_wait(empty, (it & 1) ^ 1)) { atomicExch(p.err_flag, 31); ok = false; break; }
          if (rank == 0) mbar_expect_tx(full, 2 * (kABytes + bcols * KS * 2));
          uint8_t* sa = stage;
          uint8_t* sb = stage + kABytes;
#pragma unroll
          for (int c = 0; c < BM / 64; ++c)
            tma_load_2d_pair(sa + c * CHUNK_BYTES, tmA, full_leader, un.m0 + rank * BM + c * 64, a_row + kb * KS, pol);
          for (int c = 0; c < bcols / 64; ++c)
            tma_load_2d_pair(sb + c * CHUNK_BYTES, tmB, full_leader, un.n0 + rank * bcols + c * 64, b_row + kb * KS, pol);
        }
      }
    }
  } else if (warp == 1) {
    // ---- MMA issuer (leader CTA) -----------------------------------------------------------------
    if (rank == 0 && elect_one()) {
      int it = 0;
      bool ok = true;
      for (int n = 0; n < my_units && ok; ++n) {
        const int buf = n & 1;
        const uint32_t idesc = n < p.full_rounds ? IDESC_FULL : IDESC_STRIP;
        if (!mbar_wait(&tmem_empty[buf], ((n >> 1) & 1) ^ 1)) { atomicExch(p.err_flag, 32); break; }
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * PN);
        for (int kb = 0; kb < num_kb; ++kb, ++it) {
          if (!mbar_wait(full, it & 1)) { atomicExch(p.err_flag, 33); ok = false; break; }
          tc_fence_after_sync();
          const uint32_t a_addr = smem_u32(stage);
          const uint32_t b_addr = a_addr + kABytes;
#pragma unroll
          for (int k = 0; k < KS / MMA_K; ++k) {
            const uint32_t adv = k * MMA_K * KB_BYTES;
            const uint64_t da = make_smem_desc(a_addr + adv, CHUNK_BYTES, 1024, kSwizzle128B);
            const uint64_t db = make_smem_desc(b_addr + adv, CHUNK_BYTES, 1024, kSwizzle128B);
            mma_bf16_pair(d_tmem, da, db, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          mma_commit_pair(empty);
        }
        if (ok) mma_commit_pair(&tmem_full[buf]);
      }
    }
  } else if (warp >= 4) {
    // ---- update warps: as in tc_update_kernel, on this CTA's 128 rows of the unit ----------------------
    // Eight of them: a warp can only read the 32 tensor-memory lanes of its quarter (warp index mod 4), so
    // two warps share every quarter and take the even / the odd 32-column blocks of a unit, each with its
    // own ring of R / 2 slots.  One warp per quarter spent most of its time in its own issue latencies
    // (shared-memory round trips, copy issue) with the data already waiting; two per scheduler hide them.
    static_assert(R % 2 == 0, "the ring is split between two warps");
    constexpr int R2 = R / 2;
    const int q = warp & 3, half = (warp - 4) >> 2;
    uint8_t* my_ring = ring_base + (half * 4 + q) * R2 * kSlotBytes;
    uint64_t* my_full = wv_full + (half * 4 + q) * R2;
    // this warp's chunks: every second 32-column block of every unit, in order
    const int my_chunks = p.full_rounds * (PN / 64) + my_strips * (PN / 128);
    const uint32_t tmem_empty_leader = map_to_rank(smem_u32(tmem_empty), 0);

    // the loader walks the unit list on its own, one decode per unit
    int ld_j = 0, ld_n = 0, ld_c = half;
    PUnit ld_un = decode_punit(p, 0, pb, pairs);
    auto load_next = [&]() {
      if (ld_j >= my_chunks) return;
      int y = ld_un.m0 + rank * BM + q * 32, x = ld_un.n0 + ld_c * 32;
      block_coords(p.layer[ld_un.layer].blocked, p.layer[ld_un.layer].N, x, y);
      uint8_t* slot = my_ring + (ld_j % R2) * kSlotBytes;
      mbar_expect_tx(&my_full[ld_j % R2], has_v ? kSlotBytes : kSlotBytes / 2);
      const int z = p.shared_state ? 0 : ld_un.g;
      tma_load_3d(slot, &maps.wl[ld_un.layer], &my_full[ld_j % R2], x, y, z);
      if (has_v) tma_load_3d(slot + kSlotBytes / 2, &maps.vl[ld_un.layer], &my_full[ld_j % R2], x, y, z);
      ++ld_j;
      ld_c += 2;
      if (ld_c >= ld_un.nc) {
        ld_c = half;
        if (++ld_n < my_units) ld_un = decode_punit(p, ld_n, pb, pairs);
      }
    };
    if (lane == 0)
      for (int j = 0; j < R2; ++j) load_next();

    const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
    bool ok = true;
    int j = 0;
    for (int n = 0; n < my_units && ok; ++n) {
      const PUnit un = decode_punit(p, n, pb, pairs);
      const int g = un.g, m0 = un.m0 + rank * BM, n0 = un.n0;
      const int ldw = p.layer[un.layer].N;
      __nv_bfloat16* Wb = p.layer[un.layer].Wb;
      const int buf = n & 1;
      ok = __all_sync(0xffffffffu, mbar_wait(&tmem_full[buf], (n >> 1) & 1));
      if (!ok) { if (lane == 0) atomicExch(p.err_flag, 34); break; }
      tc_fence_after_sync();
#pragma unroll 1
      for (int ci = half; ci < un.nc; ci += 2, ++j) {
        uint8_t* slot = my_ring + (j % R2) * kSlotBytes;
        uint32_t r[32];
        tmem_ld_32x32(taddr + buf * PN + ci * 32, r);
        ok = __all_sync(0xffffffffu, mbar_wait(&my_full[j % R2], (j / R2) & 1));
        tmem_ld_wait();
        if (ci + 2 >= un.nc) {
          // this warp's part of the accumulator has been read: tell the leader's MMA warp (16 arrivals, the
          // eight update warps of both CTAs, free the buffer)
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(tmem_empty_leader + (uint32_t)(buf * 8));
        }
        if (!ok) { if (lane == 0) atomicExch(p.err_flag, 35); break; }
        const int64_t at = (int64_t)g * p.w_gstride + copy_index(p.layer[un.layer].pM, ldw, m0 + q * 32 + lane, n0 + ci * 32);
        uint32_t cp[8];
#pragma unroll
        for (int jj = 0; jj < 8; ++jj) {
          const int off = lane * 128 + ((jj ^ (lane & 7)) << 4);
          float4 w = *reinterpret_cast<float4*>(slot + off);
          float ws[4] = {w.x, w.y, w.z, w.w};
          float vs[4] = {0.f, 0.f, 0.f, 0.f};
          if (has_v) {
            const float4 v = *reinterpret_cast<float4*>(slot + kSlotBytes / 2 + off);
            vs[0] = v.x; vs[1] = v.y; vs[2] = v.z; vs[3] = v.w;
          }
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float gr = __uint_as_float(r[jj * 4 + e]);
            const float step = has_v ? fmaf(p.mu, vs[e], gr) : gr;
            vs[e] = step;
            ws[e] = fmaf(-p.lr, step, ws[e]);
          }
          *reinterpret_cast<float4*>(slot + off) = make_float4(ws[0], ws[1], ws[2], ws[3]);
          if (has_v) *reinterpret_cast<float4*>(slot + kSlotBytes / 2 + off) = make_float4(vs[0], vs[1], vs[2], vs[3]);
          if (Wb != nullptr) {
            __nv_bfloat162 lo = __floats2bfloat162_rn(ws[0], ws[1]);
            __nv_bfloat162 hi = __floats2bfloat162_rn(ws[2], ws[3]);
            cp[(jj & 3) * 2] = *reinterpret_cast<uint32_t*>(&lo);
            cp[(jj & 3) * 2 + 1] = *reinterpret_cast<uint32_t*>(&hi);
            if ((jj & 3) == 3) st_global_v8(Wb + at + (jj - 3) * 4, cp);
          }
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          int y = m0 + q * 32, x = n0 + ci * 32;
          block_coords(p.layer[un.layer].blocked, ldw, x, y);
          tma_store_3d(&maps.w[un.layer], slot, x, y, g);
          if (has_v) tma_store_3d(&maps.v[un.layer], slot + kSlotBytes / 2, x, y, g);
          bulk_commit();
          bulk_wait_read<1>();
          if (j >= 1) load_next();
        }
        __syncwarp();
      }
    }
    if (lane == 0) bulk_wait_all();
    tc_fence_before_sync();
  }
  // neither CTA leaves while the other may still read its operands or signal its barriers
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc_pair(tmem_base, 2 * PN);
  }
}

// ---- one local step of every replica AND the averaging step, from a synchronized start ------------------------
// With a communication period of 1 (where AdaComm ends up for most of a long run, Section 4.2) every local step
// starts with all m replicas holding the same W and v, and ends with the average of the m updated replicas
// (Section 2, PASGD update rule, k mod tau = 0).  Done as update-then-average, that is: read W, v of m replicas,
// write them, read them again, write the mean m times.  Here a CTA owns a 128 x 64 block of W for ALL replicas:
//   * the old block (W, v) comes in once, from the synchronized copy, and stays in shared memory;
//   * for g = 0 .. m-1 the tensor core forms G_g = dZ_g^T A_g for the block (two accumulators in tensor memory, so
//     the products of replica g+1 overlap the arithmetic of replica g), and the update warps form
//     v_g = mu v + G_g, w_g = w - lr v_g exactly as the update kernel would and add them, in replica order, to
//     running sums kept in registers (one thread: one row, 32 columns, both sums);
//   * after the last replica the sums are divided by (float)m and the mean goes out to all m replicas, their bf16
//     copies and the synchronized copy.
// The arithmetic per element is that of tc_update_kernel followed by average_kernel (same fused multiply-adds,
// same order of the m additions, one division), so the state is the same bit for bit; the per-replica values are
// never written.  Traffic: 8 m + 2 m + 16 bytes per parameter instead of 2 * (16 m + 2 m).
// Eight update warps: warp w reads tensor-memory lanes 32 (w mod 4).., the two warps of a quarter take the
// left / right 32 columns.
constexpr int SN = 64;                  // columns of a unit
constexpr int kSyncThreads = 384;
constexpr int kSyncStages = 4;          // operand stages of 64 mini-batch rows: one replica's products ahead (the
                                        // tensor core waited for operands 70 % of the time with three)
struct SLayer {
  int N, n_tiles, tile_begin;           // row length of W, units per row block, first unit of the layer
  const int64_t* b_row_off;
  __nv_bfloat16* Wb;
  float *W, *V;                         // master weights / momentum of replica 0 (replica stride w_gstride)
  float *Ws, *Vs;                       // the same tensors in the synchronized copy
  int blocked;
  int pM;                               // as in ULayer
};
struct SParams {
  SLayer layer[kMaxLayers];
  int n_layers, total_units;
  int K, groups, rows_per_group;
  float lr, mu;
  int64_t w_gstride;
  int* err_flag;
};
struct SSmem {
  static constexpr int kStageBytes = (BM + SN) * kRowsBf16 * 2;        // dZ tile + layer-input tile, 64 rows
  static constexpr int kOperandBytes = kSyncStages * kStageBytes;
  static constexpr int kBaseBytes = 8 * kSlotBytes;                    // 8 blocks of 32 x 32 (W and v) = the unit
  static constexpr int kBars = 2 * kSyncStages + 4 + 3 * 2 * 8;
  static constexpr int kTotal = 1024 + kOperandBytes + 2 * kBaseBytes + kBars * 8 + 16;
  static_assert(kTotal <= 227 * 1024, "shared memory budget");
};
struct SUnit { int layer, m0, n0; };
__device__ __forceinline__ SUnit decode_sunit(const SParams& p, int u) {
  int l = 0;
#pragma unroll
  for (int i = 1; i < kMaxLayers; ++i)
    if (i < p.n_layers && u >= p.layer[i].tile_begin) l = i;
  const int r = u - p.layer[l].tile_begin, nt = p.layer[l].n_tiles;
  return SUnit{l, (r / nt) * BM, (r % nt) * SN};
}

// The mean of one 32 x 32 block (W at `slot`, v 4 KB behind it, 128-byte rows with XOR-swizzled 16-byte pieces) goes
// out to every replica, to the bf16 copies and to the synchronized copy with plain 16-byte stores, eight lanes to a
// 128-byte row.  The block is read from shared memory once; after_read() runs when it is in registers.
template <typename F>
__device__ __forceinline__ void store_mean_block(const SParams& p, const SLayer& ly, const SUnit& un, int q, int half,
                                                 const uint8_t* slot, int m, bool has_v, int lane, F after_read) {
  const int row0 = lane >> 3, piece = lane & 7;
  const int64_t ldw = ly.N;
  float4 w4[8], v4[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int row = i * 4 + row0;
    w4[i] = *reinterpret_cast<const float4*>(slot + row * 128 + ((piece ^ (row & 7)) << 4));
    if (has_v) v4[i] = *reinterpret_cast<const float4*>(slot + kSlotBytes / 2 + row * 128 + ((piece ^ (row & 7)) << 4));
  }
  after_read();
  uint2 cp[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(w4[i].x, w4[i].y);
    __nv_bfloat162 hi = __floats2bfloat162_rn(w4[i].z, w4[i].w);
    cp[i] = make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
  }
  // where this lane's first row piece goes, and the distance to its next one (four rows down): row-major,
  // or inside the block's own 4 KB when the master copy is blocked; the bf16 copy row-major or in panels
  const int64_t rm = (int64_t)(un.m0 + q * 32 + row0) * ldw + un.n0 + half * 32 + piece * 4;
  const int64_t mat = ly.blocked ? ((int64_t)((un.m0 >> 5) + q) * (ldw >> 5) + (un.n0 >> 5) + half) * 1024 +
                                       row0 * 32 + piece * 4
                                 : rm;
  const int64_t mstep = ly.blocked ? 4 * 32 : 4 * ldw;
  const int64_t at = copy_index(ly.pM, (int)ldw, un.m0 + q * 32 + row0, un.n0 + half * 32 + piece * 4);
  const int64_t bstep = ly.pM ? 4 * 64 : 4 * ldw;
  for (int g = 0; g <= m; ++g) {
    // g = m: the synchronized copy
    float* Wd = (g < m ? ly.W + (int64_t)g * p.w_gstride : ly.Ws) + mat;
    float* Vd = (g < m ? ly.V + (int64_t)g * p.w_gstride : ly.Vs) + mat;
#pragma unroll
    for (int i = 0; i < 8; ++i) *reinterpret_cast<float4*>(Wd + i * mstep) = w4[i];
    if (has_v) {
#pragma unroll
      for (int i = 0; i < 8; ++i) *reinterpret_cast<float4*>(Vd + i * mstep) = v4[i];
    }
    if (ly.Wb != nullptr && g < m) {
      __nv_bfloat16* Bd = ly.Wb + (int64_t)g * p.w_gstride + at;
#pragma unroll
      for (int i = 0; i < 8; ++i) *reinterpret_cast<uint2*>(Bd + i * bstep) = cp[i];
    }
  }
}

// SHARED: every replica enters with the synchronized W and v (a period of 1).  Otherwise (the last step of a longer
// period) replica g's own block comes in for every g, through the two buffers of each update warp in turn, and the
// update warps send the mean out themselves: the buffers have no room for a block that waits for a store warp.
template <bool SHARED>
__global__ void __launch_bounds__(kSyncThreads, 1)
tc_sync_step_kernel(const __grid_constant__ UMaps maps, const __grid_constant__ SParams p) {
  using L = SSmem;
  constexpr int KS = kRowsBf16, MMA_K = 16, STAGES = kSyncStages;
  constexpr int CHUNK_BYTES = KS * KB_BYTES;
  constexpr int kABytes = BM * KS * 2;
  constexpr uint32_t IDESC = make_idesc(1u, true, true, BM, SN);

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* stage_base = smem;
  uint8_t* base_buf = smem + L::kOperandBytes;                 // [2][8 blocks][W 4 KB | v 4 KB]
  uint64_t* full = reinterpret_cast<uint64_t*>(base_buf + 2 * L::kBaseBytes);
  uint64_t* empty = full + STAGES;
  uint64_t* tmem_full = empty + STAGES;       // [2]
  uint64_t* tmem_empty = tmem_full + 2;       // [2]
  uint64_t* base_full = tmem_empty + 2;       // [2][8]: the old block of update warp i of buffer b has arrived
  uint64_t* mean_ready = base_full + 16;      // [2][8]: update warp i has left the mean of its block in buffer b
  uint64_t* mean_gone = mean_ready + 16;      // [2][8]: the stores of that block have read shared memory
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(mean_gone + 16);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_kb = p.K / KS;
  const int bx = blockIdx.x, grid = gridDim.x;
  const int my_units = bx < p.total_units ? (p.total_units - 1 - bx) / grid + 1 : 0;
  const int m = p.groups;
  const bool has_v = p.mu != 0.f;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&tmem_full[b], 1); mbar_init(&tmem_empty[b], 8); }
    for (int i = 0; i < 48; ++i) mbar_init(&base_full[i], 1);        // base_full, mean_ready, mean_gone
    fence_mbar_init();
    for (int l = 0; l < p.n_layers; ++l) {
      prefetch_tmap(&maps.a[l]); prefetch_tmap(&maps.b[l]); prefetch_tmap(&maps.w[l]); prefetch_tmap(&maps.v[l]);
      prefetch_tmap(&maps.wl[l]); prefetch_tmap(&maps.vl[l]);
    }
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, 2 * SN);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  grid_dep_wait();
  grid_dep_launch();

  if (warp == 0) {
    // ---- operand producer: for every unit, the tiles of replica 0, 1, ... in turn ----------------------------
    if (elect_one()) {
      const uint64_t pol = l2_policy(2);
      int it = 0;
      bool ok = true;
      for (int n = 0; n < my_units && ok; ++n) {
        const SUnit un = decode_sunit(p, bx + n * grid);
        const CUtensorMap* tmA = &maps.a[un.layer];
        const CUtensorMap* tmB = &maps.b[un.layer];
        const int64_t* b_off = p.layer[un.layer].b_row_off;
        for (int g = 0; g < m && ok; ++g) {
          const int a_row = g * p.rows_per_group;
          const int b_row = b_off ? (int)b_off[g] : a_row;
          for (int kb = 0; kb < num_kb; ++kb, ++it) {
            const int s = it % STAGES;
            if (!mbar_wait(&empty[s], ((it / STAGES) & 1) ^ 1)) { atomicExch(p.err_flag, 51); ok = false; break; }
            mbar_expect_tx(&full[s], L::kStageBytes);
            uint8_t* sa = stage_base + s * L::kStageBytes;
            issue_mn_tile<64, KS>(sa, tmA, &full[s], un.m0, BM, a_row + kb * KS, pol);
            issue_mn_tile<64, KS>(sa + kABytes, tmB, &full[s], un.n0, SN, b_row + kb * KS, pol);
          }
        }
      }
    }
  } else if (warp == 1) {
    // ---- MMA issuer ----------------------------------------------------------------------------------------
    if (elect_one()) {
      int it = 0;
      bool ok = true;
      const int total_acc = my_units * m;
      for (int a = 0; a < total_acc && ok; ++a) {
        const int buf = a & 1;
        if (!mbar_wait(&tmem_empty[buf], ((a >> 1) & 1) ^ 1)) { atomicExch(p.err_flag, 52); break; }
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * SN);
        for (int kb = 0; kb < num_kb; ++kb, ++it) {
          const int s = it % STAGES;
          if (!mbar_wait(&full[s], (it / STAGES) & 1)) { atomicExch(p.err_flag, 53); ok = false; break; }
          tc_fence_after_sync();
          const uint32_t a_addr = smem_u32(stage_base + s * L::kStageBytes);
          const uint32_t b_addr = a_addr + kABytes;
#pragma unroll
          for (int k = 0; k < KS / MMA_K; ++k) {
            const uint32_t adv = k * MMA_K * KB_BYTES;
            const uint64_t da = make_smem_desc(a_addr + adv, CHUNK_BYTES, 1024, kSwizzle128B);
            const uint64_t db = make_smem_desc(b_addr + adv, CHUNK_BYTES, 1024, kSwizzle128B);
            mma_bf16(d_tmem, da, db, IDESC, (kb | k) != 0 ? 1u : 0u);
          }
          mma_commit(&empty[s]);
        }
        if (ok) mma_commit(&tmem_full[buf]);
      }
    }
  } else if (warp == 2 || warp == 3) {
    // ---- store warps: one per column half.  The mean of a block goes out to every replica, to the bf16 copies
    // and to the synchronized copy with plain 16-byte stores, eight lanes to a 128-byte row, from registers: the
    // block is read from shared memory once and its buffer is free at once.  These warps wait for memory, not
    // for arithmetic, so they run beside the update warps, which are already working on the next unit; and the
    // bulk-copy engine stays free for the operand tiles (with the mean leaving through it as well, the products
    // waited behind the queued stores: 5.6 k cycles per replica against 2 k).
    const int half = warp - 2;
    bool ok = true;
    for (int n = 0; SHARED && n < my_units && ok; ++n) {
      const SUnit un = decode_sunit(p, bx + n * grid);
      const SLayer& ly = p.layer[un.layer];
      for (int q = 0; q < 4 && ok; ++q) {
        const int wi = half * 4 + q;
        const uint8_t* slot = base_buf + (n & 1) * L::kBaseBytes + wi * kSlotBytes;
        ok = __all_sync(0xffffffffu, mbar_wait(&mean_ready[(n & 1) * 8 + wi], (n >> 1) & 1));
        if (!ok) { if (lane == 0) atomicExch(p.err_flag, 57); break; }
        // once the block is in registers its buffer is released (the arrival orders the reads before it)
        store_mean_block(p, ly, un, q, half, slot, m, has_v, lane, [&] {
          __syncwarp();
          if (lane == 0) mbar_arrive(&mean_gone[(n & 1) * 8 + wi]);
        });
      }
    }
  } else if (warp >= 4) {
    // ---- update warps ------------------------------------------------------------------------------------------
    const int q = warp & 3, half = (warp - 4) >> 2, wi = half * 4 + q;
    const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(half * 32);
    const float mf = (float)m;
    if (!SHARED) {
      // ---- every replica's own W, v: block of accumulator a = n m + g in buffer a & 1 ---------------------------
      const int total = my_units * m;
      auto load_rep = [&](int a) {           // lane 0
        const int n = a / m, g = a - n * m;
        const SUnit un = decode_sunit(p, bx + n * grid);
        uint8_t* slot = base_buf + (a & 1) * L::kBaseBytes + wi * kSlotBytes;
        uint64_t* bar = &base_full[(a & 1) * 8 + wi];
        mbar_expect_tx(bar, has_v ? kSlotBytes : kSlotBytes / 2);
        int x = un.n0 + half * 32, y = un.m0 + q * 32;
        block_coords(p.layer[un.layer].blocked, p.layer[un.layer].N, x, y);
        tma_load_3d(slot, &maps.w[un.layer], bar, x, y, g);
        if (has_v) tma_load_3d(slot + kSlotBytes / 2, &maps.v[un.layer], bar, x, y, g);
      };
      if (lane == 0 && total > 0) load_rep(0);
      bool ok = true;
      int a = 0;
      for (int n = 0; n < my_units && ok; ++n) {
        const SUnit un = decode_sunit(p, bx + n * grid);
        float sw[32], sv[32];
#pragma unroll 1
        for (int g = 0; g < m; ++g, ++a) {
          const int buf = a & 1;
          uint8_t* slot = base_buf + buf * L::kBaseBytes + wi * kSlotBytes;
          // the other buffer was last read by this warp (replica a - 1, or the mean of the unit before): refill it
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0 && a + 1 < total) load_rep(a + 1);
          ok = __all_sync(0xffffffffu, mbar_wait(&base_full[buf * 8 + wi], (a >> 1) & 1));
          if (!ok) { if (lane == 0) atomicExch(p.err_flag, 58); break; }
          ok = __all_sync(0xffffffffu, mbar_wait(&tmem_full[buf], (a >> 1) & 1));
          if (!ok) { if (lane == 0) atomicExch(p.err_flag, 55); break; }
          tc_fence_after_sync();
          uint32_t r[32];
          tmem_ld_32x32(taddr + buf * SN, r);
          tmem_ld_wait();
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&tmem_empty[buf]);
#pragma unroll
          for (int jj = 0; jj < 8; ++jj) {
            const int off = lane * 128 + ((jj ^ (lane & 7)) << 4);
            const float4 w = *reinterpret_cast<const float4*>(slot + off);
            const float ws[4] = {w.x, w.y, w.z, w.w};
            float vs[4] = {0.f, 0.f, 0.f, 0.f};
            if (has_v) {
              const float4 v = *reinterpret_cast<const float4*>(slot + kSlotBytes / 2 + off);
              vs[0] = v.x; vs[1] = v.y; vs[2] = v.z; vs[3] = v.w;
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float gr = __uint_as_float(r[jj * 4 + e]);
              const float step = has_v ? fmaf(p.mu, vs[e], gr) : gr;          // v_g
              const float wn = fmaf(-p.lr, step, ws[e]);                     // w_g
              sw[jj * 4 + e] = g == 0 ? wn : __fadd_rn(sw[jj * 4 + e], wn);
              sv[jj * 4 + e] = g == 0 ? step : __fadd_rn(sv[jj * 4 + e], step);
            }
          }
        }
        if (!ok) break;
        // the mean takes the place of the last replica's block (its buffer is not refilled before the next
        // iteration), and this warp sends it out
        uint8_t* slot = base_buf + ((a - 1) & 1) * L::kBaseBytes + wi * kSlotBytes;
#pragma unroll
        for (int e = 0; e < 32; ++e) { sw[e] = __fdiv_rn(sw[e], mf); sv[e] = __fdiv_rn(sv[e], mf); }
        __syncwarp();
#pragma unroll
        for (int jj = 0; jj < 8; ++jj) {
          const int off = lane * 128 + ((jj ^ (lane & 7)) << 4);
          *reinterpret_cast<float4*>(slot + off) = make_float4(sw[jj * 4], sw[jj * 4 + 1], sw[jj * 4 + 2], sw[jj * 4 + 3]);
          if (has_v)
            *reinterpret_cast<float4*>(slot + kSlotBytes / 2 + off) =
                make_float4(sv[jj * 4], sv[jj * 4 + 1], sv[jj * 4 + 2], sv[jj * 4 + 3]);
        }
        __syncwarp();
        store_mean_block(p, p.layer[un.layer], un, q, half, slot, m, has_v, lane, [] {});
      }
      tc_fence_before_sync();
    } else {
    auto load_base = [&](int n) {            // lane 0: this warp's 32 x 32 block of the old W and v of unit n
      const SUnit un = decode_sunit(p, bx + n * grid);
      uint8_t* slot = base_buf + (n & 1) * L::kBaseBytes + wi * kSlotBytes;
      uint64_t* bar = &base_full[(n & 1) * 8 + wi];
      mbar_expect_tx(bar, has_v ? kSlotBytes : kSlotBytes / 2);
      int x = un.n0 + half * 32, y = un.m0 + q * 32;
      block_coords(p.layer[un.layer].blocked, p.layer[un.layer].N, x, y);
      tma_load_3d(slot, &maps.wl[un.layer], bar, x, y, 0);
      if (has_v) tma_load_3d(slot + kSlotBytes / 2, &maps.vl[un.layer], bar, x, y, 0);
    };
    if (lane == 0 && my_units > 0) load_base(0);
    bool ok = true;
    int a = 0;                                // accumulators consumed so far
    for (int n = 0; n < my_units && ok; ++n) {
      const SUnit un = decode_sunit(p, bx + n * grid);
      uint8_t* slot = base_buf + (n & 1) * L::kBaseBytes + wi * kSlotBytes;
      const int ldw = p.layer[un.layer].N;
      __nv_bfloat16* Wb = p.layer[un.layer].Wb;
      float sw[32], sv[32];
      ok = __all_sync(0xffffffffu, mbar_wait(&base_full[(n & 1) * 8 + wi], (n >> 1) & 1));
      if (!ok) { if (lane == 0) atomicExch(p.err_flag, 54); break; }
#pragma unroll 1
      for (int g = 0; g < m; ++g, ++a) {
        const int buf = a & 1;
        ok = __all_sync(0xffffffffu, mbar_wait(&tmem_full[buf], (a >> 1) & 1));
        if (!ok) { if (lane == 0) atomicExch(p.err_flag, 55); break; }
        tc_fence_after_sync();
        uint32_t r[32];
        tmem_ld_32x32(taddr + buf * SN, r);
        tmem_ld_wait();
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(&tmem_empty[buf]);
        // halfway through a unit the stores of the unit before have normally left shared memory: its buffer
        // takes the old block of the next unit
        if (g == m / 2 && n + 1 < my_units) {
          if (n >= 1) {
            ok = __all_sync(0xffffffffu, mbar_wait(&mean_gone[((n + 1) & 1) * 8 + wi], (((n + 1) >> 1) - 1) & 1));
            if (!ok) { if (lane == 0) atomicExch(p.err_flag, 56); break; }
          }
          if (lane == 0) load_base(n + 1);
        }
#pragma unroll
        for (int jj = 0; jj < 8; ++jj) {
          const int off = lane * 128 + ((jj ^ (lane & 7)) << 4);
          const float4 w = *reinterpret_cast<const float4*>(slot + off);
          const float ws[4] = {w.x, w.y, w.z, w.w};
          float vs[4] = {0.f, 0.f, 0.f, 0.f};
          if (has_v) {
            const float4 v = *reinterpret_cast<const float4*>(slot + kSlotBytes / 2 + off);
            vs[0] = v.x; vs[1] = v.y; vs[2] = v.z; vs[3] = v.w;
          }
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float gr = __uint_as_float(r[jj * 4 + e]);
            const float step = has_v ? fmaf(p.mu, vs[e], gr) : gr;          // v_g
            const float wn = fmaf(-p.lr, step, ws[e]);                     // w_g
            // the mean's sum, in replica order: s = x^(0); s = s + x^(g)
            sw[jj * 4 + e] = g == 0 ? wn : __fadd_rn(sw[jj * 4 + e], wn);
            sv[jj * 4 + e] = g == 0 ? step : __fadd_rn(sv[jj * 4 + e], step);
          }
        }
      }
      if (!ok) break;
      // the mean, into the block's place in shared memory, and from there to every replica and the synchronized copy
#pragma unroll
      for (int e = 0; e < 32; ++e) { sw[e] = __fdiv_rn(sw[e], mf); sv[e] = __fdiv_rn(sv[e], mf); }
#pragma unroll
      for (int jj = 0; jj < 8; ++jj) {
        const int off = lane * 128 + ((jj ^ (lane & 7)) << 4);
        *reinterpret_cast<float4*>(slot + off) = make_float4(sw[jj * 4], sw[jj * 4 + 1], sw[jj * 4 + 2], sw[jj * 4 + 3]);
        if (has_v)
          *reinterpret_cast<float4*>(slot + kSlotBytes / 2 + off) =
              make_float4(sv[jj * 4], sv[jj * 4 + 1], sv[jj * 4 + 2], sv[jj * 4 + 3]);
      }
      // hand the block to the store warp of this column half and go on with the next unit
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(&mean_ready[(n & 1) * 8 + wi]);
    }
    tc_fence_before_sync();
    }
  }
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, 2 * SN);
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

template <bool TF32, int STAGES, int R, int KS>
int launch_update(const TcUpdateArgs* layers, int n, cudaStream_t st) {
  using L = USmem<TF32, STAGES, R, KS>;
  auto kern = tc_update_kernel<TF32, STAGES, R, KS>;
  static uint64_t configured = 0;        // one bit per device
  {
    cudaError_t e = allow_dynamic_smem(kern, (int)(L::kTotal), &configured);
    if (e != cudaSuccess) return e;
  }
  const TcUpdateArgs& a0 = layers[0];
  UParams p{};
  UMaps maps;
  int total = 0;
  bool shared = true;
  for (int i = 0; i < n; ++i) shared = shared && layers[i].mapWsync != nullptr && layers[i].mapVsync != nullptr;
  for (int i = 0; i < n; ++i) {
    const TcUpdateArgs& a = layers[i];
    ULayer& l = p.layer[i];
    l.N = a.N;
    l.n_tiles = a.N / BN;
    l.tiles_per_group = (a.M / BM) * (a.N / BN);
    l.tile_begin = total;
    l.b_row_off = a.row_off;
    l.Wb = a.Wb;
    l.blocked = a.blocked ? 1 : 0;
    l.pM = a.panel ? a.M : 0;
    total += l.tiles_per_group * a.groups;
    maps.a[i] = *a.maps.a; maps.b[i] = *a.maps.b; maps.w[i] = *a.mapW; maps.v[i] = *a.mapV;
    maps.wl[i] = shared ? *a.mapWsync : *a.mapW; maps.vl[i] = shared ? *a.mapVsync : *a.mapV;
  }
  for (int i = n; i < kMaxLayers; ++i) {     // unused slots hold valid descriptors
    maps.a[i] = maps.a[0]; maps.b[i] = maps.b[0]; maps.w[i] = maps.w[0]; maps.v[i] = maps.v[0];
    maps.wl[i] = maps.wl[0]; maps.vl[i] = maps.vl[0];
  }
  p.n_layers = n; p.total_tiles = total;
  {
    const int ctas = total < num_sms() ? total : num_sms();
    p.full_rounds = total / ctas;
    p.tail_units = (total - p.full_rounds * ctas) * (TF32 ? 4 : 2);
  }
  p.K = a0.B; p.groups = a0.groups; p.rows_per_group = a0.B; p.shared_state = shared ? 1 : 0;
  p.lr = a0.lr; p.mu = a0.mu; p.w_gstride = a0.w_gstride; p.err_flag = a0.err_flag;
  const int grid = total < num_sms() ? total : num_sms();
  return launch_dep(kern, dim3(grid), dim3(kThreads), L::kTotal, st, 1, maps, p);
}

template <int R, int KS>
int launch_update_pair(const TcUpdateArgs* layers, int n, cudaStream_t st) {
  using L = USmem<false, 1, R, KS>;
  auto kern = tc_update_pair_kernel<R, KS>;
  static uint64_t configured = 0;        // one bit per device
  {
    cudaError_t e = allow_dynamic_smem(kern, (int)(L::kTotal), &configured);
    if (e != cudaSuccess) return e;
  }
  const TcUpdateArgs& a0 = layers[0];
  PParams p{};
  UMaps maps;
  int total = 0;
  bool shared = true;
  for (int i = 0; i < n; ++i) shared = shared && layers[i].mapWsync != nullptr && layers[i].mapVsync != nullptr;
  for (int i = 0; i < n; ++i) {
    const TcUpdateArgs& a = layers[i];
    PLayer& l = p.layer[i];
    l.N = a.N;
    l.n_tiles = a.N / PN;
    l.tiles_per_group = (a.M / 256) * (a.N / PN);
    l.tile_begin = total;
    l.b_row_off = a.row_off;
    l.Wb = a.Wb;
    l.blocked = a.blocked ? 1 : 0;
    l.pM = a.panel ? a.M : 0;
    total += l.tiles_per_group * a.groups;
    maps.a[i] = *a.maps.a; maps.b[i] = *a.maps.b; maps.w[i] = *a.mapW; maps.v[i] = *a.mapV;
    maps.wl[i] = shared ? *a.mapWsync : *a.mapW; maps.vl[i] = shared ? *a.mapVsync : *a.mapV;
  }
  for (int i = n; i < kMaxLayers; ++i) {
    maps.a[i] = maps.a[0]; maps.b[i] = maps.b[0]; maps.w[i] = maps.w[0]; maps.v[i] = maps.v[0];
    maps.wl[i] = maps.wl[0]; maps.vl[i] = maps.vl[0];
  }
  const int max_pairs = num_sms() / 2;
  const int pairs = total < max_pairs ? total : max_pairs;
  p.n_layers = n;
  p.full_rounds = total / pairs;
  p.tail_units = (total - p.full_rounds * pairs) * 2;
  p.K = a0.B; p.rows_per_group = a0.B; p.groups = a0.groups; p.shared_state = shared ? 1 : 0;
  p.lr = a0.lr; p.mu = a0.mu; p.w_gstride = a0.w_gstride; p.err_flag = a0.err_flag;
  return launch_dep(kern, dim3(2 * pairs), dim3(kPairThreads), L::kTotal, st, 2, maps, p);
}

}  // namespace

bool tc_update_shape_ok(bool fp32, int M, int N, int B) {
  return M > 0 && N > 0 && B > 0 && M % BM == 0 && N % BN == 0 && B % (fp32 ? 32 : 64) == 0;
}

bool tc_sync_step_shape_ok(bool fp32, int M, int N, int B) {
  return !fp32 && M > 0 && N > 0 && B > 0 && M % BM == 0 && N % SN == 0 && B % kRowsBf16 == 0;
}

// layers[0..n): with the synchronized-copy descriptors (mapWsync / mapVsync) on every layer the replicas are taken to
// enter synchronized and the old state is read from that copy; without them every replica's own state is read
int launch_tc_sync_step(const TcUpdateArgs* layers, int n, cudaStream_t st, int64_t* launches) {
  if (n < 1 || n > kMaxLayers) return cudaErrorInvalidValue;
  bool shared = true;
  for (int i = 0; i < n; ++i) {
    if (layers[i].fp32 || layers[i].W == nullptr || layers[i].V == nullptr || layers[i].Wsync == nullptr ||
        layers[i].Vsync == nullptr)
      return cudaErrorInvalidValue;
    shared = shared && layers[i].mapWsync != nullptr && layers[i].mapVsync != nullptr;
  }
  static uint64_t configured[2] = {0, 0};
  {
    cudaError_t e = shared ? allow_dynamic_smem(tc_sync_step_kernel<true>, (int)SSmem::kTotal, &configured[0])
                           : allow_dynamic_smem(tc_sync_step_kernel<false>, (int)SSmem::kTotal, &configured[1]);
    if (e != cudaSuccess) return e;
  }
  const TcUpdateArgs& a0 = layers[0];
  SParams p{};
  UMaps maps;
  int total = 0;
  for (int i = 0; i < n; ++i) {
    const TcUpdateArgs& a = layers[i];
    SLayer& l = p.layer[i];
    l.N = a.N; l.n_tiles = a.N / SN; l.tile_begin = total; l.b_row_off = a.row_off; l.Wb = a.Wb;
    l.W = a.W; l.V = a.V; l.Ws = a.Wsync; l.Vs = a.Vsync; l.blocked = a.blocked ? 1 : 0;
    l.pM = a.panel ? a.M : 0;
    total += (a.M / BM) * (a.N / SN);
    maps.a[i] = *a.maps.a; maps.b[i] = *a.maps.b; maps.w[i] = *a.mapW; maps.v[i] = *a.mapV;
    maps.wl[i] = shared ? *a.mapWsync : *a.mapW; maps.vl[i] = shared ? *a.mapVsync : *a.mapV;
  }
  for (int i = n; i < kMaxLayers; ++i) {
    maps.a[i] = maps.a[0]; maps.b[i] = maps.b[0]; maps.w[i] = maps.w[0]; maps.v[i] = maps.v[0];
    maps.wl[i] = maps.wl[0]; maps.vl[i] = maps.vl[0];
  }
  p.n_layers = n; p.total_units = total;
  p.K = a0.B; p.groups = a0.groups; p.rows_per_group = a0.B;
  p.lr = a0.lr; p.mu = a0.mu; p.w_gstride = a0.w_gstride; p.err_flag = a0.err_flag;
  if (launches) ++*launches;
  const int grid = total < num_sms() ? total : num_sms();
  if (shared) return launch_dep(tc_sync_step_kernel<true>, dim3(grid), dim3(kSyncThreads), SSmem::kTotal, st, 1, maps, p);
  return launch_dep(tc_sync_step_kernel<false>, dim3(grid), dim3(kSyncThreads), SSmem::kTotal, st, 1, maps, p);
}

int tc_update_max_layers() { return kMaxLayers; }
int tc_update_box_rows(bool fp32) { return fp32 ? kRowsFp32 : kRowsBf16; }

// layers[0..n): same batch, replica count, rates and element type; the largest layer should come first
int launch_tc_update(const TcUpdateArgs* layers, int n, cudaStream_t st, int64_t* launches) {
  if (n < 1 || n > kMaxLayers) return cudaErrorInvalidValue;
  if (launches) ++*launches;
  if (layers[0].fp32) return launch_update<true, 5, 4, kRowsFp32>(layers, n, st);
  // bf16 layers that are multiples of 256 in both directions: the CTA-pair kernel
  bool pair = layers[0].allow_pair;
  for (int i = 0; i < n; ++i) pair = pair && layers[i].M % 256 == 0 && layers[i].N % PN == 0;
  if (pair) return launch_update_pair<6, kRowsBf16>(layers, n, st);
  return launch_update<false, 1, 6, kRowsBf16>(layers, n, st);
}

}  // namespace ls
