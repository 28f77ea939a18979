// Internal declarations shared by the translation units of libls.so.
// Nothing here is part of the C ABI (see include/ls.h for that).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdlib.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

#include "ls.h"

namespace ls {

constexpr int kRowOffCap = 512;        // local steps per offsets upload
constexpr int kEvalCap = 8192;         // mini-batch chunks per ls_eval_loss call
constexpr int64_t kAlignFloats = 64;   // every tensor and every replica starts on a 256-byte boundary

// Where everything lives.  Offsets inside one replica are in elements (the
// same for the fp32 master copy, the momentum buffer and the operand copy);
// offsets inside the state block are in bytes.
//
// Operand copies.  bf16 models keep a bf16 rounding of the weights; whoever writes the weights writes
// the copy.  fp32 models need none: the tensor-core kernels split every fp32 operand tile into its
// tf32 upper part and the remainder in shared memory (see gemm_tc.cu).
struct Layout {
  int L = 0;
  int dims[LS_MAX_LAYERS + 1] = {0};
  int has_bias = 0;
  int bf16 = 0;
  int m = 0;
  int batch = 0;
  int max_width = 0;                   // max(dims[1..L])
  int64_t P = 0;                       // interface parameter count
  int64_t stride = 0;                  // elements between replicas (padded)
  int64_t w_off[LS_MAX_LAYERS] = {0};  // padded offsets inside a replica
  int64_t b_off[LS_MAX_LAYERS] = {0};
  int64_t w_flat[LS_MAX_LAYERS] = {0}; // offsets in the flat interface layout
  int64_t b_flat[LS_MAX_LAYERS] = {0};
  size_t params_off = 0, mom_off = 0;
  size_t shadow_off = 0;                     // bf16 [m][stride] copy of the weights (bf16 models)
  size_t act_off[LS_MAX_LAYERS + 1] = {0};   // post-ReLU activations = inputs of layers 1..L-1
  size_t dz_off[LS_MAX_LAYERS] = {0};        // dZ_l = gradient w.r.t. the output of layer l, [m][batch][dims[l+1]]
  size_t logits_off = 0;                     // [m][batch][dims[L]] fp32
  size_t dzl_off = 0;                        // fp32 dZ of a narrow output layer [m][batch][dims[L]]
  size_t rowloss_off = 0;                    // per-sample losses [LS_MAX_REPLICAS][batch]
  size_t headcnt_off = 0;                    // per-replica CTA counters of the output-layer kernel
  size_t headpart_off = 0;                   // partial logits of a fused output layer [m][parts][batch][16]
  size_t rowoff_off = 0;                     // int64 [kRowOffCap][m]
  size_t evaloff_off = 0;                    // int64 [kEvalCap]
  size_t evalloss_off = 0;                   // float [kEvalCap]
  size_t stage_x_off[2] = {0, 0};            // [m][batch][dims[0]] input staging for host batches
  size_t stage_y_off[2] = {0, 0};            // [m][batch] labels / targets
  size_t stage_loss_off = 0;                 // float [kRowOffCap][m]
  size_t err_off = 0;                        // int: device-side error flag (bounded waits that ran out)
  size_t anchor_off = 0, blocku_off = 0;     // block momentum: period-start model and global buffer, [stride] each
  int tiled[LS_MAX_LAYERS] = {0};            // W_l (and v_l) stored as 32 x 32 blocks, see TileMap
  int panel[LS_MAX_LAYERS] = {0};            // the bf16 copy of W_l stored as 64-column panels, see TileMap
  size_t retile_off = 0;                     // staging for one matrix in row-major order (host <-> tiled layout)
  size_t hstep_off = 0, hstep_cnt_off = 0;   // scratch and counters of the one-launch output layer (head_step.cu)
  size_t sync_off = 0;                       // synchronized copy: [2][stride] parameters and momentum as every replica
                                             // held them right after the last averaging step
  size_t total = 0;
};

int make_layout(int m, const ls_model_spec* spec, int batch, Layout* out);

// Blocked storage of the streamed weight matrices.  The fp32 master copy (and momentum) of a matrix that the
// streaming update kernels own is not kept row by row but as 32 x 32 blocks, each block 4 KB of consecutive
// memory, blocks in row-major order of (row block, column block): element (r, c) of an M x N matrix sits at
//     ((r / 32) * (N / 32) + c / 32) * 1024 + (r % 32) * 32 + c % 32 .
// The update kernels move exactly such blocks, so every bulk copy of theirs is one contiguous 4 KB run instead of
// 32 pieces of 128 bytes a row pitch apart, which DRAM serves markedly better (measured on the update of the
// bf16 workload: 785 -> 734 us).  Everything element-wise (averaging, partial sums, the synchronized copy, block
// momentum) is indifferent to the order.  The host interface (ls_set_params, ls_get_state, ...) is row-major:
// copy_replica retiles.
//
// The bf16 operand copy of such a matrix, which only the tensor-core GEMMs read, is kept in panels of 64
// columns (128 bytes, the width of one operand box): panel p holds columns [64 p, 64 p + 64) of all rows, row after
// row, so element (r, c) sits at
//     (c / 64) * M * 64 + r * 64 + c % 64 .
// An operand box (64 columns x 64 rows) is then 8 KB of consecutive memory for both GEMMs, and what an update warp
// writes for a 32 x 32 block (32 rows x 64 bytes) stays inside 4 KB instead of being spread over 32 rows of the
// matrix.  The GEMMs address it as a 4-D tensor [replica][panel][row][64] (tc_make_panel_map).  Matrices that a
// CUDA-core GEMM may read keep a row-major copy (panel = 0).  Whoever writes the copy from the master's element
// order finds the place with shadow_index().
struct TileMap {
  int n = 0;
  int64_t begin[LS_MAX_LAYERS] = {0};   // first element of the matrix inside a replica vector
  int64_t size[LS_MAX_LAYERS] = {0};    // rows * cols
  int cols[LS_MAX_LAYERS] = {0};
  int panel[LS_MAX_LAYERS] = {0};       // bf16 copy in 64-column panels (else row-major)
};
// Index, in the bf16 operand copy of a replica vector, of element e of the master's arrangement: the panel
// arrangement for matrices kept that way, row-major otherwise.  Eight consecutive e starting at a multiple of 8
// stay consecutive.
__host__ __device__ inline int64_t shadow_index(const TileMap& t, int64_t e) {
  for (int j = 0; j < t.n; ++j) {
    const int64_t local = e - t.begin[j];
    if (local >= 0 && local < t.size[j]) {
      const int64_t blk = local >> 10;
      const int r = (int)(local >> 5) & 31, c = (int)local & 31, nb = t.cols[j] >> 5;
      const int64_t rb = blk / nb, cb = blk - rb * nb;
      const int64_t row = rb * 32 + r, col = cb * 32 + c;
      if (!t.panel[j]) return t.begin[j] + row * t.cols[j] + col;
      const int64_t rows = t.size[j] / t.cols[j];
      return t.begin[j] + (col >> 6) * rows * 64 + row * 64 + (col & 63);
    }
  }
  return e;
}

}  // namespace ls

// TMA descriptors of the tensors the tensor-core kernels read (built once per handle).
struct alignas(64) TcMaps {
  CUtensorMap w[LS_MAX_LAYERS];                           // weights as operands, 3-D [replica][out][in]
  CUtensorMap act[LS_MAX_LAYERS];                         // input of layer l >= 1, 2-D [m*batch][dims[l]]
  CUtensorMap dz[LS_MAX_LAYERS];                          // dZ_l, 2-D [m*batch][dims[l+1]]
  CUtensorMap x_data;                                     // bound dataset, 2-D [n_rows][dims[0]]
  CUtensorMap x_stage[2];                                 // staging buffers of host batches
  CUtensorMap wf[LS_MAX_LAYERS], vf[LS_MAX_LAYERS];       // fp32 master weights / momentum, 32 x 32 blocks
  CUtensorMap wsync[LS_MAX_LAYERS], vsync[LS_MAX_LAYERS]; // the same blocks of the synchronized copy (one vector each)
};

struct ls_handle {
  TcMaps maps;       // for K-major reads (and every read of a bf16 tensor)
  TcMaps maps_mn;    // fp32 models: the same tensors for MN-major reads (swizzle in 32-byte units)
  TcMaps maps_upd;   // dz / act / x_* as the update kernel reads them (MN-major, boxes of tc_update_box_rows rows)
  uint32_t magic;
  ls::Layout lay;
  ls_model_spec spec;
  float lr, mu;
  char* state;
  cudaStream_t stream;
  cudaStream_t copy_stream;
  cudaEvent_t ev_copied[2], ev_consumed[2];
  const void* x_dev;
  const void* y_dev;
  int64_t n_rows;
  int last_cuda;
  bool allow_pair;        // CTA-pair kernels enabled (see pair_kernels_enabled)
  bool allow_head_step;   // one-launch output layer enabled (see head_step_enabled)
  ls::TileMap tiles;      // the blocked matrices of a replica vector
  bool sync_valid;        // every replica's parameters and momentum equal the synchronized copy, bit for bit
  // replicas spread over several GPUs (ls_set_shard): this handle holds m of m_total replicas
  int shard_G, shard_m_total;
  float* shard_partial;   // [n_buf][stride] this GPU's partial sums
  float* shard_gathered;  // [G][n_buf][stride] every GPU's partial sums, in rank order
  ls_exchange_fn shard_fn;
  void* shard_ctx;
  int64_t launches;
  float* pinned;          // small pinned host scratch (eval losses)
  // per-kernel timing (ls_profile_begin / ls_profile_end)
  uint32_t prof_mask;
  int prof_layer;
  int prof_used;
  int prof_cap;
  cudaEvent_t* prof_ev;   // 2 events per record
  int16_t* prof_tag;      // class * LS_MAX_LAYERS + layer per record
};

namespace ls {

constexpr uint32_t kMagic = 0x4c53474du;

// ---- programmatic dependent launch ------------------------------------------------------------
// Every kernel of the step is launched with programmatic stream serialization: its CTAs may become
// resident while the kernel before it in the stream is still draining, run their prologue (barrier
// setup, tensor-memory allocation, descriptor prefetch) and then block in grid_dep_wait() until that
// kernel has completed and its writes are visible.  No kernel touches global memory before the wait,
// so the results are those of plain stream order; only launch latency and prologues overlap.
#ifdef __CUDACC__
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... P, typename... A>
inline cudaError_t launch_dep(void (*kern)(P...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              unsigned cluster_x, A&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  unsigned n = 0;
  // LS_DISABLE_PDL=1 in the environment launches every kernel in plain stream order (a diagnostic switch)
  static const bool pdl = [] { const char* e = getenv("LS_DISABLE_PDL"); return !(e && e[0] == '1'); }();
  if (pdl) {
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  if (cluster_x > 1) {       // the CTAs that share an output tile form one cluster along x
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = cluster_x;
    attr[n].val.clusterDim.y = 1;
    attr[n].val.clusterDim.z = 1;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<P>(args)...);
}
#endif

// LS_DISABLE_PAIR=1 in the environment keeps every launch of a handle on the one-CTA tensor-core kernels (a
// diagnostic switch; read once, when the handle is created, and carried in the launch arguments).
// LS_DISABLE_HEAD_STEP=1 in the environment at ls_create time: the output layer of a training step runs as the
// forward kernel followed by head_bwd_kernel instead of the one-launch kernel (a diagnostic switch; the tests
// compare the two).
inline bool head_step_enabled() {
  const char* e = getenv("LS_DISABLE_HEAD_STEP");
  return !(e && e[0] == '1');
}
inline bool pair_kernels_enabled() {
  const char* e = getenv("LS_DISABLE_PAIR");
  return !(e && e[0] == '1');
}

// cudaFuncAttributeMaxDynamicSharedMemorySize is a per-device attribute of a kernel: set it once per device
// (`done` is a per-kernel bit mask over the device ordinals, kept by the caller in a function-local static).
template <typename K>
inline cudaError_t allow_dynamic_smem(K kern, int bytes, uint64_t* done) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const uint64_t bit = 1ull << (dev & 63);
  if (*done & bit) return cudaSuccess;
  e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) *done |= bit;
  return e;
}

inline float* params_of(const ls_handle* h) { return reinterpret_cast<float*>(h->state + h->lay.params_off); }
inline float* mom_of(const ls_handle* h) { return reinterpret_cast<float*>(h->state + h->lay.mom_off); }
inline __nv_bfloat16* shadow_of(const ls_handle* h) {
  return h->lay.bf16 ? reinterpret_cast<__nv_bfloat16*>(h->state + h->lay.shadow_off) : nullptr;
}
inline float* anchor_of(const ls_handle* h) { return reinterpret_cast<float*>(h->state + h->lay.anchor_off); }
inline float* blocku_of(const ls_handle* h) { return reinterpret_cast<float*>(h->state + h->lay.blocku_off); }
inline float* sync_of(const ls_handle* h) { return reinterpret_cast<float*>(h->state + h->lay.sync_off); }

// ---- averaging (average.cu) ---------------------------------------------
// n_buf buffers of m vectors each; buffer b starts at base + b*buf_stride floats,
// vector j of it at + j*stride.  shadow (optional, same strides) receives the
// bf16 rounding of the mean of buffer 0.  Returns a cudaError_t.
// bm (optional, n_buf == 1): block momentum, see average.cu; anchor and u are vectors of n floats.
struct BlockMomentum {
  float* anchor;
  float* u;
  float lr, beta;
};
// sync_out (optional): the mean of buffer b is also written to sync_out + b*sync_stride (the synchronized copy;
// sync_stride 0 means n).
int launch_average(float* base, int n_buf, int64_t buf_stride, int m, int64_t n, int64_t stride,
                   __nv_bfloat16* shadow, cudaStream_t st, int64_t* launches,
                   const BlockMomentum* bm = nullptr, float* sync_out = nullptr, int64_t sync_stride = 0,
                   const TileMap* tiles = nullptr);    // tiles: the blocked matrices of `base` (`shadow`: shadow_index)

// The same for n_pieces short pieces [begin[r], begin[r] + len[r]) of the replica vectors that lie outside every
// blocked matrix, in one launch when their ends fall on multiples of 8 floats (else one launch each).
int launch_average_pieces(float* base, int n_buf, int64_t buf_stride, int m, const int64_t* begin, const int64_t* len,
                          int n_pieces, int64_t stride, __nv_bfloat16* shadow, cudaStream_t st, int64_t* launches,
                          float* sync_out, int64_t sync_stride);

// ---- averaging over several GPUs (shard_average.cu) -------------------------
// out[b] = sum over the m vectors of buffer b in index order; then, with the G partial sums of every GPU
// gathered in rank order (vector g of buffer b at parts + g*part_stride + b*part_buf_stride), the mean
// (p_0 + ... + p_{G-1}) / m_total written to the m_local replicas of every buffer (and the bf16 copy of buffer 0).
int launch_partial_sum(const float* base, int n_buf, int64_t buf_stride, int m, int64_t n, int64_t stride, float* out,
                       int64_t out_stride, cudaStream_t st, int64_t* launches);
int launch_combine(const float* parts, int G, int64_t part_stride, int64_t part_buf_stride, int m_total, int64_t n,
                   float* base, int n_buf, int64_t buf_stride, int m_local, int64_t stride, __nv_bfloat16* shadow,
                   cudaStream_t st, int64_t* launches, const TileMap* tiles = nullptr);

// ---- fp32-accumulate CUDA-core grouped GEMMs (gemm_simt.cu) ---------------
struct FwdArgs {           // Z = A W^T + b, optional ReLU
  const void* A;           // [groups][M][K] (or dataset rows through row_off)
  const int64_t* row_off;  // device, per group first row of A; null: group g starts at g*M
  const void* W;           // weight matrix of group 0, [N][K]
  int64_t w_gstride;       // elements between groups' weights (0: shared)
  const float* bias;       // fp32 master bias of group 0 or null
  int64_t bias_gstride;
  void* C;                 // [groups][M][N]
  int M, N, K, groups;
  int relu;
};
struct DxArgs {            // dZ_prev = (dZ W) * 1[act > 0]
  const void* dZ;          // [groups][M][K]
  const void* W;           // [K][N]
  int64_t w_gstride;
  const void* act;         // [groups][M][N] post-ReLU activation of the previous layer
  void* C;                 // [groups][M][N]
  int M, N, K, groups;
};
struct DwArgs {            // G = dZ^T A ; v = mu v + G ; W -= lr v ; operand copy of W
  const void* dZ;          // [groups][B][M]
  const void* A;           // [groups][B][N] (or dataset rows through row_off)
  const int64_t* row_off;
  float* W;                // fp32 master [M][N] of group 0
  float* V;                // momentum, same layout (unused when mu == 0)
  __nv_bfloat16* Wb;       // bf16 copy or null
  int64_t w_gstride;
  int M, N, B, groups;
  float lr, mu;
};
int launch_fwd(const FwdArgs& a, bool a_bf16, bool w_bf16, bool c_bf16, cudaStream_t st, int64_t* launches);
int launch_dx(const DxArgs& a, bool bf16, cudaStream_t st, int64_t* launches);
int launch_dw(const DwArgs& a, bool bf16, cudaStream_t st, int64_t* launches);

// ---- loss, dZ_L, bias update (loss.cu) ------------------------------------
struct LossArgs {
  const float* logits;     // [groups][B][C]
  const void* y;           // int32 labels or float targets of the bound rows
  const int64_t* row_off;  // device, per group first row in y
  void* dZ;                // [groups][B][C] or null (forward only)
  float* loss_out;         // [groups] or null
  int B, C, groups;
  int loss_kind;
};
int launch_loss(const LossArgs& a, bool dz_bf16, cudaStream_t st, int64_t* launches);

struct BiasArgs {          // gb = colsum(dZ); v = mu v + gb; b -= lr v
  const void* dZ;          // [groups][B][N]
  float* bias;
  float* vbias;
  int64_t gstride;
  int B, N, groups;
  float lr, mu;
};
int launch_bias(const BiasArgs& a, bool bf16, cudaStream_t st, int64_t* launches);

// ---- small linear models: all local steps of a call in one launch (period_linear.cu) -------------------
bool linear_period_ok(int B, int K, int C, bool has_v);
int launch_linear_period(const float* X, const void* y, const int64_t* row_off, float* W, float* V, float* bias,
                         float* vbias, int64_t gstride, float* loss_out, int tau, int m, int B, int K, int C, int kind,
                         float lr, float mu, cudaStream_t st, int64_t* launches);

// ---- narrow output layer (head.cu) ---------------------------------------------
struct HeadFwdArgs {
  const void* A; const int64_t* a_row_off;   // layer input [groups][B][K] (or dataset rows)
  const float* W; int64_t w_gstride; const float* bias;
  const void* y; const int64_t* y_row_off;
  float* dZ;                                 // [groups][B][C] or null (forward only)
  float* row_loss; float* loss_out; unsigned int* counters;
  int B, C, K, groups, loss_kind;
  int defer_loss;                            // 1: only write row_loss; the backward kernel forms loss_out
};
struct HeadBwdArgs {
  const void* A; const int64_t* a_row_off;
  const float* dZ;
  float* W; float* V; __nv_bfloat16* Wb; float* bias; float* vbias; int64_t w_gstride;
  void* dPrev;                               // dZ of the layer below [groups][B][K] or null
  float* pbias; float* pvbias;               // bias / its momentum of the layer below (updated from the column
                                             // sums of dPrev) or null; replica stride w_gstride
  const float* row_loss; float* loss_out;    // row losses left by the forward kernel and where their mean goes, or null
  int B, C, K, groups;
  float lr, mu;
};
// The output layer of a training step in one launch (head_step.cu): what launch_head_fwd (want dZ) followed by
// launch_head_bwd compute, for bf16 layer inputs [groups][B][K] of a 10-class softmax layer.
struct HeadStepArgs {
  const void* A;                             // layer input, bf16, group g at row g*B
  const void* y; const int64_t* y_row_off;   // int32 labels; first row of group g
  float* W; float* V; __nv_bfloat16* Wb; float* bias; float* vbias; int64_t w_gstride;
  void* dPrev;                               // dZ of the layer below [groups][B][K], bf16
  float* pbias; float* pvbias;               // bias / its momentum of the layer below, or null
  float* loss_out;                           // [groups] mini-batch mean loss, or null
  float* scratch;                            // head_step_scratch_bytes(groups, C, K) bytes, contents irrelevant
  unsigned int* counters;                    // head_step_counter_bytes(groups) bytes, zero before the first launch
  int B, C, K, groups, loss_kind;
  float lr, mu;
};
size_t head_step_scratch_bytes(int m, int C, int K);
size_t head_step_counter_bytes(int m);
bool head_step_ok(const HeadStepArgs& a);
int launch_head_step(const HeadStepArgs& a, cudaStream_t st, int64_t* launches);
bool head_shape_ok(int B, int C);
int launch_head_fwd(const HeadFwdArgs& a, bool a_bf16, cudaStream_t st, int64_t* launches);
int launch_head_bwd(const HeadBwdArgs& a, bool a_bf16, cudaStream_t st, int64_t* launches);

// fp32 -> bf16 copy of n elements (refresh of the weight copies)
// m vectors of `stride` elements each; tiles: the matrices that src holds blocked (dst: shadow_index)
int launch_to_bf16(const float* src, __nv_bfloat16* dst, int m, int64_t stride, const TileMap* tiles, cudaStream_t st,
                   int64_t* launches);
// one matrix between row-major and blocked order (to_blocked: dst blocked <- src row-major, else the reverse)
int launch_retile(float* dst, const float* src, int rows, int cols, bool to_blocked, cudaStream_t st, int64_t* launches);

// ---- tcgen05 grouped GEMMs (gemm_tc.cu) -------------------------------------
int tc_make_map_2d(CUtensorMap* out, const void* base, bool fp32, bool mn32, int64_t rows, int64_t cols);
int tc_make_map_2d_rows(CUtensorMap* out, const void* base, bool fp32, bool mn32, int64_t rows, int64_t cols,
                        int box_rows);
int tc_make_map_3d(CUtensorMap* out, const void* base, bool fp32, bool mn32, int64_t rows, int64_t cols,
                   int64_t groups, int64_t gstride);
int tc_make_block_map_3d(CUtensorMap* out, const void* base, int64_t rows, int64_t cols, int64_t groups,
                         int64_t gstride, bool blocked = false);
// 4-D map over the bf16 copies of `groups` matrices [rows][cols] kept in 64-column panels (see TileMap):
// dimensions (64, rows, cols / 64, groups); a box is 64 columns x 64 rows, read at (0, row, column / 64, group)
int tc_make_panel_map(CUtensorMap* out, const void* base, int64_t rows, int64_t cols, int64_t groups, int64_t gstride);
bool tc_shape_ok(bool fp32, int M, int N, int K);   // output rows, output columns, contraction length
struct TcOperandMaps {
  const CUtensorMap *a, *b;
};
// A narrow output layer evaluated by the forward kernel of the layer before it (W null: none).
struct TcHead {
  const float* W; int64_t w_gstride; const float* bias;    // [C][N] fp32 master weights, bias or null
  const void* y; const int64_t* y_row_off;                 // labels / targets and each group's first row
  float* part;               // scratch [groups][parts][M][16] partial logits, parts <= tc_fwd_head_parts(N)
  unsigned int* counters;    // [groups], zero before the launch, zero again after it
  float* dZ;                 // [groups][M][C] or null (forward only)
  float* row_loss;           // [groups][M]
  float* loss_out;           // [groups] or null
  int C, kind, defer_loss;   // defer_loss: leave the mean of the row losses to the backward kernel
};
bool tc_fwd_fuses_head(bool fp32, int M, int N, int C);
int tc_fwd_head_parts(int N);
struct TcFwdArgs {
  TcOperandMaps maps;        // a: [rows][K] input (dataset rows through row_off, else group g at row g*M); b: weights
  bool fp32;
  const int64_t* row_off;
  int w_z0, w_zstep;         // replica used by group g = w_z0 + g*w_zstep
  bool w_panel = false;      // maps.b is a panel map (tc_make_panel_map)
  const float* bias; int64_t bias_gstride;
  void* C;                   // [groups][M][N] bf16 or fp32
  const CUtensorMap* c_map;  // bf16: C as a 2-D tensor [groups*M][N], boxes of 64 x 64 (pair kernel's stores), or null
  TcHead head;
  int M, N, K, groups, relu;
  int* err_flag;
  bool allow_pair;           // CTA-pair kernels may be chosen
};
struct TcDxArgs {
  TcOperandMaps maps;        // a: dZ_l [groups*M][K]; b: weights
  bool fp32;
  const void* act; void* C;
  const CUtensorMap* c_map;   // bf16: C and act as 2-D tensors [groups*M][N], boxes of 64 x 64, or null
  const CUtensorMap* act_map;
  int w_zstep;               // replica whose weights group g reads = g * w_zstep (0: every group reads replica 0's)
  bool w_panel = false;      // maps.b is a panel map (tc_make_panel_map)
  int M, N, K, groups;
  // bias / its momentum of the layer that produced `act` (group 0; replica stride bias_gstride): updated
  // from the column sums of C inside the kernel when tc_dx_fuses_bias(); else null
  float* bias; float* vbias; int64_t bias_gstride; float lr, mu;
  int* err_flag;
  bool allow_pair;
};
// whether launch_tc_dx can also apply the bias update (every output tile holds all M rows)
bool tc_dx_fuses_bias(bool fp32, int M, int N);
struct TcDwArgs {
  TcOperandMaps maps;        // a: dZ_l [groups*B][M]; b: layer input [rows][N]
  bool fp32;
  const int64_t* row_off;
  float* W; float* V; __nv_bfloat16* Wb; int64_t w_gstride;
  int M, N, B, groups;
  float lr, mu;
  int* err_flag;
};
// persistent streaming update kernel (update_tc.cu)
struct TcUpdateArgs {
  TcOperandMaps maps;        // a: dZ_l [groups*B][M]; b: layer input [rows][N]   (MN-major reads)
  const CUtensorMap* mapW;   // fp32 master weights [replica][M][N], 32 x 32 blocks
  const CUtensorMap* mapV;   // momentum, same shape
  // when every replica enters the step with the same W and v: descriptors of the synchronized copy (one
  // vector, [1][M][N]) that the old values are read from instead; null otherwise
  const CUtensorMap* mapWsync; const CUtensorMap* mapVsync;
  // the same four tensors as plain pointers (replica 0; replica stride w_gstride): the fused step + average
  // kernel stores through them
  float* W; float* V; float* Wsync; float* Vsync;
  bool blocked;              // W, v (and their synchronized copy) are stored as 32 x 32 blocks (TileMap)
  bool panel = false;        // Wb is kept in 64-column panels (TileMap), else row-major
  bool fp32;
  const int64_t* row_off;
  __nv_bfloat16* Wb; int64_t w_gstride;
  int M, N, B, groups;
  float lr, mu;
  int* err_flag;
  int layer;                 // which layer of the model this is (bookkeeping of the caller)
  bool allow_pair;
};
bool tc_update_shape_ok(bool fp32, int M, int N, int B);
int tc_update_max_layers();
int tc_update_box_rows(bool fp32);     // rows of the TMA boxes its operand maps (dZ, layer input) must have
// one launch for the updates of layers[0..n) (n <= tc_update_max_layers(); same batch, replicas, rates, type)
int launch_tc_update(const TcUpdateArgs* layers, int n, cudaStream_t st, int64_t* launches);
// One local step of all replicas from a synchronized start, fused with the averaging step that follows it
// (communication period 1): the layers' W and v leave the launch averaged, in every replica and in the
// synchronized copy.  Same argument records; mapWsync / mapVsync are required.
bool tc_sync_step_shape_ok(bool fp32, int M, int N, int B);
int launch_tc_sync_step(const TcUpdateArgs* layers, int n, cudaStream_t st, int64_t* launches);
int launch_tc_fwd(const TcFwdArgs& a, cudaStream_t st, int64_t* launches);
int launch_tc_dx(const TcDxArgs& a, cudaStream_t st, int64_t* launches);
int launch_tc_dw(const TcDwArgs& a, cudaStream_t st, int64_t* launches);

}  // namespace ls
