// Host side of libls.so: the C ABI declared in include/ls.h, the memory layout
// of the replicas, and the launch sequence of one local step.
#include <math.h>
#include <string.h>

#include <algorithm>
#include <chrono>
#include <new>
#include <vector>

#include "ls_internal.h"
#include "tc_ptx.cuh"

using namespace ls;

namespace ls {

static inline int64_t round_up(int64_t v, int64_t a) { return (v + a - 1) / a * a; }
static inline size_t round_up_sz(size_t v, size_t a) { return (v + a - 1) / a * a; }

static int check_spec(const ls_model_spec* s) {
  if (s == nullptr) return LS_ERR_INVALID_ARG;
  if (s->n_layers < 1 || s->n_layers > LS_MAX_LAYERS) return LS_ERR_INVALID_ARG;
  for (int l = 0; l <= s->n_layers; ++l)
    if (s->dims[l] < 1 || s->dims[l] > (1 << 20)) return LS_ERR_INVALID_ARG;
  if (s->dims[s->n_layers] > LS_MAX_OUT) return LS_ERR_INVALID_ARG;
  if (s->loss != LS_LOSS_SOFTMAX_CE && s->loss != LS_LOSS_MSE_HALF) return LS_ERR_INVALID_ARG;
  if (s->loss == LS_LOSS_MSE_HALF && s->dims[s->n_layers] != 1) return LS_ERR_INVALID_ARG;
  if (s->has_bias != 0 && s->has_bias != 1) return LS_ERR_INVALID_ARG;
  if (s->gemm_dtype != LS_GEMM_FP32 && s->gemm_dtype != LS_GEMM_BF16) return LS_ERR_INVALID_ARG;
  if (s->momentum_mode < LS_MOMENTUM_AVERAGE || s->momentum_mode > LS_MOMENTUM_BLOCK) return LS_ERR_INVALID_ARG;
  if (s->momentum_mode == LS_MOMENTUM_BLOCK && !(s->block_momentum >= 0.f && s->block_momentum < 1.f))
    return LS_ERR_INVALID_ARG;
  if (!(s->weight_decay == 0.0f)) return isfinite(s->weight_decay) ? LS_ERR_UNSUPPORTED : LS_ERR_INVALID_ARG;
  return LS_OK;
}

int make_layout(int m, const ls_model_spec* spec, int batch, Layout* out) {
  int rc = check_spec(spec);
  if (rc != LS_OK) return rc;
  if (m < 1 || m > LS_MAX_REPLICAS || batch < 1 || batch > LS_MAX_BATCH || out == nullptr) return LS_ERR_INVALID_ARG;
  Layout lay;
  lay.L = spec->n_layers;
  lay.has_bias = spec->has_bias;
  lay.bf16 = spec->gemm_dtype == LS_GEMM_BF16;
  lay.m = m;
  lay.batch = batch;
  int64_t cur = 0, flat = 0;
  for (int l = 0; l <= lay.L; ++l) lay.dims[l] = spec->dims[l];
  for (int l = 0; l < lay.L; ++l) {
    const int64_t n_out = lay.dims[l + 1], n_in = lay.dims[l];
    if (n_out > lay.max_width) lay.max_width = (int)n_out;
    lay.w_off[l] = cur;
    lay.w_flat[l] = flat;
    cur = round_up(cur + n_out * n_in, kAlignFloats);
    flat += n_out * n_in;
    lay.b_off[l] = cur;
    lay.b_flat[l] = flat;
    if (lay.has_bias) {
      cur = round_up(cur + n_out, kAlignFloats);
      flat += n_out;
    }
  }
  lay.P = flat;
  lay.stride = cur;
  const size_t A = 256;
  const size_t esz = lay.bf16 ? 2 : 4;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t at = off; off = round_up_sz(off + bytes, A); return at; };
  lay.params_off = take((size_t)m * lay.stride * 4);
  lay.mom_off = take((size_t)m * lay.stride * 4);
  if (lay.bf16) lay.shadow_off = take((size_t)m * lay.stride * 2);
  for (int l = 1; l < lay.L; ++l) {
    lay.act_off[l] = take((size_t)m * batch * lay.dims[l] * esz);
  }
  for (int l = 0; l < lay.L; ++l) lay.dz_off[l] = take((size_t)m * batch * lay.dims[l + 1] * esz);
  lay.logits_off = take((size_t)m * batch * lay.dims[lay.L] * 4);
  lay.dzl_off = take((size_t)m * batch * lay.dims[lay.L] * 4);
  lay.rowloss_off = take((size_t)LS_MAX_REPLICAS * batch * 4);
  lay.headcnt_off = take((size_t)LS_MAX_REPLICAS * 4);
  if (lay.L >= 2 && head_shape_ok(batch, lay.dims[lay.L]) &&
      tc_fwd_fuses_head(!lay.bf16, batch, lay.dims[lay.L - 1], lay.dims[lay.L]))
    lay.headpart_off = take((size_t)m * tc_fwd_head_parts(lay.dims[lay.L - 1]) * batch * 16 * 4);
  if (lay.bf16 && lay.L >= 2 && lay.headpart_off == 0 && head_shape_ok(batch, lay.dims[lay.L])) {
    lay.hstep_off = take(head_step_scratch_bytes(m, lay.dims[lay.L], lay.dims[lay.L - 1]));
    lay.hstep_cnt_off = take(head_step_counter_bytes(m));
  }
  lay.rowoff_off = take((size_t)kRowOffCap * m * 8);
  lay.evaloff_off = take((size_t)kEvalCap * 8);
  lay.evalloss_off = take((size_t)kEvalCap * 4);
  for (int s = 0; s < 2; ++s) {
    lay.stage_x_off[s] = take((size_t)m * batch * lay.dims[0] * esz);
    lay.stage_y_off[s] = take((size_t)m * batch * 4);
  }
  lay.stage_loss_off = take((size_t)kRowOffCap * m * 4);
  lay.err_off = take(256);
  lay.sync_off = take((size_t)2 * lay.stride * 4);
  // bf16 models: the master copy of every matrix that the streaming update kernels own is stored in 32 x 32
  // blocks (see TileMap); fp32 models keep row-major matrices, because their GEMMs read the master copy itself
  size_t retile = 0;
  for (int l = 0; l < lay.L; ++l) {
    lay.tiled[l] = lay.bf16 && tc_update_shape_ok(false, lay.dims[l + 1], lay.dims[l], batch) ? 1 : 0;
    // the bf16 copy goes into panels when every GEMM that reads it is a tensor-core one (forward; data gradient)
    lay.panel[l] = lay.tiled[l] && l < lay.L - 1 && tc_shape_ok(false, batch, lay.dims[l + 1], lay.dims[l]) &&
                           (l == 0 || tc_shape_ok(false, batch, lay.dims[l], lay.dims[l + 1]))
                       ? 1 : 0;
    if (lay.tiled[l]) retile = std::max(retile, (size_t)lay.dims[l + 1] * lay.dims[l] * 4);
  }
  if (retile) lay.retile_off = take(retile);
  if (spec->momentum_mode == LS_MOMENTUM_BLOCK) {
    lay.anchor_off = take((size_t)lay.stride * 4);
    lay.blocku_off = take((size_t)lay.stride * 4);
  }
  lay.total = off;
  *out = lay;
  return LS_OK;
}

static inline bool ok_handle(const ls_handle* h) { return h != nullptr && h->magic == kMagic; }

static int cuda_fail(ls_handle* h, int e) {
  if (h) h->last_cuda = e;
  return LS_ERR_CUDA;
}
#define LS_CUDA(h, expr)                                 \
  do {                                                   \
    int _e = (int)(expr);                                \
    if (_e != (int)cudaSuccess) return cuda_fail(h, _e); \
  } while (0)

constexpr int kProfCap = 16384;

// Brackets one launch with a pair of events when its class/layer is being profiled.
struct ProfScope {
  ls_handle* h;
  int rec;
  ProfScope(ls_handle* h_, int cls, int layer) : h(h_), rec(-1) {
    if (!(h->prof_mask & (1u << cls))) return;
    if (h->prof_layer >= 0 && layer != h->prof_layer && cls != LS_K_LOSS && cls != LS_K_AVG) return;
    if (h->prof_used >= h->prof_cap) return;
    rec = h->prof_used++;
    h->prof_tag[rec] = (int16_t)(cls * LS_MAX_LAYERS + layer);
    cudaEventRecord(h->prof_ev[2 * rec], h->stream);
  }
  ~ProfScope() {
    if (rec >= 0) cudaEventRecord(h->prof_ev[2 * rec + 1], h->stream);
  }
};

// Refresh the bf16 operand copies of the weights (bf16 models).
static int refresh_shadow(ls_handle* h) {
  const int64_t n = (int64_t)h->lay.m * h->lay.stride;
  (void)n;
  if (h->lay.bf16)
    LS_CUDA(h, launch_to_bf16(params_of(h), shadow_of(h), h->lay.m, h->lay.stride, &h->tiles, h->stream, &h->launches));
  return LS_OK;
}

// One forward pass of `groups` mini-batches.  Group g reads rows
// [row_off[g], +batch) of x/y and uses the weights at w_base + g*w_gstride
// (w_gstride == 0: every group uses the same replica).
static inline int* err_flag_of(const ls_handle* h) { return reinterpret_cast<int*>(h->state + h->lay.err_off); }

// The device-side error flag after the stream has drained: a bounded wait that ran out inside a kernel left a
// code there.  Reports it once (LS_ERR_DEVICE_TIMEOUT) and clears it, so that the handle stays usable.
static int take_device_flag(ls_handle* h, int flag) {
  if (flag == 0) return LS_OK;
  LS_CUDA(h, cudaMemsetAsync(err_flag_of(h), 0, sizeof(int), h->stream));
  LS_CUDA(h, cudaStreamSynchronize(h->stream));
  return LS_ERR_DEVICE_TIMEOUT;
}
static int check_device_flag(ls_handle* h) {
  int flag = 0;
  LS_CUDA(h, cudaMemcpyAsync(&flag, err_flag_of(h), sizeof(int), cudaMemcpyDeviceToHost, h->stream));
  LS_CUDA(h, cudaStreamSynchronize(h->stream));
  return take_device_flag(h, flag);
}

// A kernel whose only job is to let a bounded wait run out: one thread waits, for at most `limit` clock ticks,
// on a barrier on which nobody ever arrives, then records the failure in *err_flag and returns, exactly as the
// tensor-core kernels do when one of their waits gives up.  No tensor memory, no bulk copies, nothing to drain.
__global__ void wait_timeout_selftest_kernel(int* err_flag, long long limit) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bar, 1);
    ptx::fence_mbar_init();
    if (!ptx::mbar_wait(&bar, 0, limit)) atomicExch(err_flag, 99);
  }
}

// x maps: [0] for K-major reads, [1] for MN-major reads of the mini-batch rows
struct XMaps { const CUtensorMap* k; const CUtensorMap* mn; const CUtensorMap* upd; };

// The output layer of a training step as ONE launch (head_step.cu) when its shape allows: fills `a`.  False: the
// forward kernel (stand-alone or riding on the GEMM before it) and head_bwd_kernel run instead.
static bool head_step_args(ls_handle* h, const void* y, const int64_t* row_off_dev, float* loss_out, HeadStepArgs& a) {
  const Layout& lay = h->lay;
  const int l = lay.L - 1;
  if (!h->allow_head_step || !lay.bf16 || l < 1 || lay.hstep_off == 0 || !head_shape_ok(lay.batch, lay.dims[lay.L]))
    return false;
  a.A = h->state + lay.act_off[l];
  a.y = y; a.y_row_off = row_off_dev;
  a.W = params_of(h) + lay.w_off[l]; a.V = mom_of(h) + lay.w_off[l]; a.Wb = shadow_of(h) + lay.w_off[l];
  a.bias = lay.has_bias ? params_of(h) + lay.b_off[l] : nullptr;
  a.vbias = mom_of(h) + lay.b_off[l];
  a.w_gstride = lay.stride;
  a.dPrev = h->state + lay.dz_off[l - 1];
  a.pbias = lay.has_bias ? params_of(h) + lay.b_off[l - 1] : nullptr;
  a.pvbias = mom_of(h) + lay.b_off[l - 1];
  a.loss_out = loss_out;
  a.scratch = reinterpret_cast<float*>(h->state + lay.hstep_off);
  a.counters = reinterpret_cast<unsigned int*>(h->state + lay.hstep_cnt_off);
  a.B = lay.batch; a.C = lay.dims[lay.L]; a.K = lay.dims[l]; a.groups = lay.m; a.loss_kind = h->spec.loss;
  a.lr = h->lr; a.mu = h->mu;
  return head_step_ok(a);
}

// shared_w: the groups are different replicas whose weights are known to be bitwise equal (first step after an
// averaging step): the tensor-core layers all read replica 0's operand copy, which then stays in L2.
static int forward(ls_handle* h, const void* x, XMaps xmap, const void* y, const int64_t* row_off_dev,
                   int groups, int64_t replica0, int64_t w_gstride, bool want_dz, float* loss_out,
                   bool shared_w = false) {
  const Layout& lay = h->lay;
  const bool bf = lay.bf16;
  const float* P = params_of(h) + replica0 * lay.stride;
  const __nv_bfloat16* S = bf ? shadow_of(h) + replica0 * lay.stride : nullptr;
  for (int l = 0; l < lay.L; ++l) {
    if (l == lay.L - 1 && head_shape_ok(lay.batch, lay.dims[lay.L])) {
      if (want_dz && groups == lay.m && replica0 == 0 && w_gstride == lay.stride) {
        // a training step: the kernel that local_step launches for this layer's backward pass does the forward too
        HeadStepArgs s;
        if (head_step_args(h, y, row_off_dev, loss_out, s)) return LS_OK;
      }
      // narrow output layer: product, loss and dZ in one kernel
      HeadFwdArgs a;
      a.A = (l == 0) ? x : (const void*)(h->state + lay.act_off[l]);
      a.a_row_off = (l == 0) ? row_off_dev : nullptr;
      a.W = P + lay.w_off[l]; a.w_gstride = w_gstride;
      a.bias = lay.has_bias ? P + lay.b_off[l] : nullptr;
      a.y = y; a.y_row_off = row_off_dev;
      a.dZ = want_dz ? reinterpret_cast<float*>(h->state + lay.dzl_off) : nullptr;
      a.row_loss = reinterpret_cast<float*>(h->state + lay.rowloss_off);
      a.loss_out = loss_out;
      a.counters = reinterpret_cast<unsigned int*>(h->state + lay.headcnt_off);
      a.B = lay.batch; a.C = lay.dims[lay.L]; a.K = lay.dims[l]; a.groups = groups; a.loss_kind = h->spec.loss;
      a.defer_loss = want_dz ? 1 : 0;       // a training step: the backward kernel of this layer forms the mean
      ProfScope ps(h, LS_K_FWD, l);
      LS_CUDA(h, launch_head_fwd(a, bf, h->stream, &h->launches));
      return LS_OK;
    }
    if (l < lay.L - 1 && tc_shape_ok(!bf, lay.batch, lay.dims[l + 1], lay.dims[l])) {
      TcFwdArgs t;
      t.fp32 = !bf;
      t.maps.a = (l == 0) ? xmap.k : &h->maps.act[l];
      t.maps.b = &h->maps.w[l];
      t.row_off = (l == 0) ? row_off_dev : nullptr;
      t.w_z0 = (int)replica0; t.w_zstep = (w_gstride != 0 && !shared_w) ? 1 : 0;
      t.w_panel = lay.panel[l] != 0;
      t.bias = lay.has_bias ? P + lay.b_off[l] : nullptr;
      t.bias_gstride = w_gstride;
      t.C = h->state + lay.act_off[l + 1];
      t.c_map = (bf && lay.dims[l + 1] % 8 == 0) ? &h->maps.act[l + 1] : nullptr;
      t.M = lay.batch; t.N = lay.dims[l + 1]; t.K = lay.dims[l]; t.groups = groups; t.relu = 1;
      t.err_flag = err_flag_of(h);
      t.allow_pair = h->allow_pair;
      t.head = TcHead{};
      const bool fuse_head = l == lay.L - 2 && lay.headpart_off != 0 && groups <= lay.m;
      if (fuse_head) {
        // the narrow output layer rides on this kernel: logits, per-sample losses and dZ_L
        TcHead& hd = t.head;
        hd.W = P + lay.w_off[lay.L - 1]; hd.w_gstride = w_gstride;
        hd.bias = lay.has_bias ? P + lay.b_off[lay.L - 1] : nullptr;
        hd.y = y; hd.y_row_off = row_off_dev;
        hd.part = reinterpret_cast<float*>(h->state + lay.headpart_off);
        hd.counters = reinterpret_cast<unsigned int*>(h->state + lay.headcnt_off);
        hd.dZ = want_dz ? reinterpret_cast<float*>(h->state + lay.dzl_off) : nullptr;
        hd.row_loss = reinterpret_cast<float*>(h->state + lay.rowloss_off);
        hd.loss_out = loss_out;
        hd.C = lay.dims[lay.L]; hd.kind = h->spec.loss; hd.defer_loss = want_dz ? 1 : 0;
      }
      ProfScope ps(h, LS_K_FWD, l);
      LS_CUDA(h, launch_tc_fwd(t, h->stream, &h->launches));
      if (fuse_head) return LS_OK;
      continue;
    }
    FwdArgs a;
    a.A = (l == 0) ? x : (const void*)(h->state + lay.act_off[l]);
    a.row_off = (l == 0) ? row_off_dev : nullptr;
    a.W = bf ? (const void*)(S + lay.w_off[l]) : (const void*)(P + lay.w_off[l]);
    a.w_gstride = w_gstride;
    a.bias = lay.has_bias ? P + lay.b_off[l] : nullptr;
    a.bias_gstride = w_gstride;
    const bool last = (l == lay.L - 1);
    a.C = last ? (void*)(h->state + lay.logits_off) : (void*)(h->state + lay.act_off[l + 1]);
    a.M = lay.batch; a.N = lay.dims[l + 1]; a.K = lay.dims[l]; a.groups = groups;
    a.relu = last ? 0 : 1;
    ProfScope ps(h, LS_K_FWD, l);
    LS_CUDA(h, launch_fwd(a, bf, bf, bf && !last, h->stream, &h->launches));
  }
  LossArgs la;
  la.logits = reinterpret_cast<const float*>(h->state + lay.logits_off);
  la.y = y; la.row_off = row_off_dev;
  la.dZ = want_dz ? (void*)(h->state + lay.dz_off[lay.L - 1]) : nullptr;
  la.loss_out = loss_out;
  la.B = lay.batch; la.C = lay.dims[lay.L]; la.groups = groups; la.loss_kind = h->spec.loss;
  ProfScope ps(h, LS_K_LOSS, 0);
  LS_CUDA(h, launch_loss(la, bf, h->stream, &h->launches));
  return LS_OK;
}

// One local update of all m replicas (forward, backward, fused SGD-momentum).
static int average(ls_handle* h);

// avg_after: this is the last local step of a period; the replicas leave the call averaged (Section 2, PASGD
// update rule, k mod tau = 0).
static int local_step(ls_handle* h, const void* x, XMaps xmap, const void* y, const int64_t* row_off_dev,
                      float* loss_out, bool avg_after = false) {
  const Layout& lay = h->lay;
  const bool bf = lay.bf16;
  const TcMaps& mn = bf ? h->maps : h->maps_mn;     // descriptors for MN-major reads
  const bool shared_w = h->sync_valid;
  int rc = forward(h, x, xmap, y, row_off_dev, lay.m, 0, lay.stride, true, loss_out, shared_w);
  if (rc != LS_OK) return rc;
  bool bias_done[LS_MAX_LAYERS] = {false};     // bias l already updated by the kernel that produced dZ_l
  // Weight updates that run on the streaming tensor-core kernel are collected and launched together after
  // the last data gradient: they are independent of one another, and dZ_l / the layer inputs stay in place.
  TcUpdateArgs upd[LS_MAX_LAYERS];
  int n_upd = 0;
  for (int l = lay.L - 1; l >= 0; --l) {
    void* dZ = h->state + lay.dz_off[l];
    if (l == lay.L - 1 && head_shape_ok(lay.batch, lay.dims[lay.L])) {
      HeadStepArgs s;
      if (head_step_args(h, y, row_off_dev, loss_out, s)) {
        // forward, loss, both gradients, update and the bias of the layer below in one launch
        if (s.pbias != nullptr) bias_done[l - 1] = true;
        ProfScope ps(h, LS_K_DW, l);
        LS_CUDA(h, launch_head_step(s, h->stream, &h->launches));
        continue;
      }
      // narrow output layer: both gradients, the update and the bias in one pass over its input
      HeadBwdArgs a;
      a.A = (l == 0) ? x : (const void*)(h->state + lay.act_off[l]);
      a.a_row_off = (l == 0) ? row_off_dev : nullptr;
      a.dZ = reinterpret_cast<const float*>(h->state + lay.dzl_off);
      a.W = params_of(h) + lay.w_off[l]; a.V = mom_of(h) + lay.w_off[l];
      a.Wb = bf ? shadow_of(h) + lay.w_off[l] : nullptr;
      a.bias = lay.has_bias ? params_of(h) + lay.b_off[l] : nullptr;
      a.vbias = mom_of(h) + lay.b_off[l];
      a.w_gstride = lay.stride;
      a.dPrev = (l > 0) ? (void*)(h->state + lay.dz_off[l - 1]) : nullptr;
      a.pbias = (l > 0 && lay.has_bias) ? params_of(h) + lay.b_off[l - 1] : nullptr;
      a.pvbias = mom_of(h) + (l > 0 ? lay.b_off[l - 1] : 0);
      if (a.pbias != nullptr) bias_done[l - 1] = true;
      a.row_loss = reinterpret_cast<const float*>(h->state + lay.rowloss_off);
      a.loss_out = loss_out;
      a.B = lay.batch; a.C = lay.dims[lay.L]; a.K = lay.dims[l]; a.groups = lay.m;
      a.lr = h->lr; a.mu = h->mu;
      ProfScope ps(h, LS_K_DW, l);
      LS_CUDA(h, launch_head_bwd(a, bf, h->stream, &h->launches));
      continue;
    }
    if (l > 0 && tc_shape_ok(!bf, lay.batch, lay.dims[l], lay.dims[l + 1])) {
      // the data gradient reads W_l before the update below overwrites it
      TcDxArgs t;
      t.fp32 = !bf;
      t.maps.a = &h->maps.dz[l];
      t.maps.b = &mn.w[l];
      t.act = h->state + lay.act_off[l];
      t.C = h->state + lay.dz_off[l - 1];
      t.c_map = (bf && lay.dims[l] % 8 == 0) ? &h->maps.dz[l - 1] : nullptr;
      t.act_map = (bf && lay.dims[l] % 8 == 0) ? &h->maps.act[l] : nullptr;
      t.M = lay.batch; t.N = lay.dims[l]; t.K = lay.dims[l + 1]; t.groups = lay.m;
      t.w_zstep = shared_w ? 0 : 1;
      t.w_panel = lay.panel[l] != 0;
      t.bias = nullptr; t.vbias = nullptr; t.bias_gstride = lay.stride; t.lr = h->lr; t.mu = h->mu;
      if (lay.has_bias && tc_dx_fuses_bias(!bf, t.M, t.N)) {
        t.bias = params_of(h) + lay.b_off[l - 1];
        t.vbias = mom_of(h) + lay.b_off[l - 1];
        bias_done[l - 1] = true;
      }
      t.err_flag = err_flag_of(h);
      t.allow_pair = h->allow_pair;
      ProfScope ps(h, LS_K_DX, l);
      LS_CUDA(h, launch_tc_dx(t, h->stream, &h->launches));
    } else if (l > 0) {
      DxArgs d;
      d.dZ = dZ;
      d.W = bf ? (const void*)(shadow_of(h) + lay.w_off[l]) : (const void*)(params_of(h) + lay.w_off[l]);
      d.w_gstride = lay.stride;
      d.act = h->state + lay.act_off[l];
      d.C = h->state + lay.dz_off[l - 1];
      d.M = lay.batch; d.N = lay.dims[l]; d.K = lay.dims[l + 1]; d.groups = lay.m;
      ProfScope ps(h, LS_K_DX, l);
      LS_CUDA(h, launch_dx(d, bf, h->stream, &h->launches));
    }
    if (tc_update_shape_ok(!bf, lay.dims[l + 1], lay.dims[l], lay.batch)) {
      TcUpdateArgs& t = upd[n_upd++];
      t.fp32 = !bf;
      t.maps.a = &h->maps_upd.dz[l];
      t.maps.b = (l == 0) ? xmap.upd : &h->maps_upd.act[l];
      t.mapW = &h->maps.wf[l];
      t.mapV = &h->maps.vf[l];
      // every replica still holds the synchronized model (first local step after an averaging step): the old
      // W and v are read once, from the synchronized copy, instead of once per replica
      t.mapWsync = h->sync_valid ? &h->maps.wsync[l] : nullptr;
      t.mapVsync = h->sync_valid ? &h->maps.vsync[l] : nullptr;
      t.W = params_of(h) + lay.w_off[l]; t.V = mom_of(h) + lay.w_off[l];
      t.Wsync = sync_of(h) + lay.w_off[l]; t.Vsync = sync_of(h) + lay.stride + lay.w_off[l];
      t.blocked = lay.tiled[l] != 0;
      t.panel = lay.panel[l] != 0;
      t.row_off = (l == 0) ? row_off_dev : nullptr;
      t.Wb = bf ? shadow_of(h) + lay.w_off[l] : nullptr;
      t.w_gstride = lay.stride;
      t.M = lay.dims[l + 1]; t.N = lay.dims[l]; t.B = lay.batch; t.groups = lay.m;
      t.lr = h->lr; t.mu = h->mu;
      t.err_flag = err_flag_of(h);
      t.layer = l;
      t.allow_pair = h->allow_pair;
    } else if (tc_shape_ok(!bf, lay.dims[l + 1], lay.dims[l], lay.batch)) {
      TcDwArgs t;
      t.fp32 = !bf;
      t.maps.a = &mn.dz[l];
      t.maps.b = (l == 0) ? xmap.mn : &mn.act[l];
      t.row_off = (l == 0) ? row_off_dev : nullptr;
      t.W = params_of(h) + lay.w_off[l];
      t.V = mom_of(h) + lay.w_off[l];
      t.Wb = bf ? shadow_of(h) + lay.w_off[l] : nullptr;
      t.w_gstride = lay.stride;
      t.M = lay.dims[l + 1]; t.N = lay.dims[l]; t.B = lay.batch; t.groups = lay.m;
      t.lr = h->lr; t.mu = h->mu;
      t.err_flag = err_flag_of(h);
      ProfScope ps(h, LS_K_DW, l);
      LS_CUDA(h, launch_tc_dw(t, h->stream, &h->launches));
    } else {
    DwArgs w;
    w.dZ = dZ;
    w.A = (l == 0) ? x : (const void*)(h->state + lay.act_off[l]);
    w.row_off = (l == 0) ? row_off_dev : nullptr;
    w.W = params_of(h) + lay.w_off[l];
    w.V = mom_of(h) + lay.w_off[l];
    w.Wb = bf ? shadow_of(h) + lay.w_off[l] : nullptr;
    w.w_gstride = lay.stride;
    w.M = lay.dims[l + 1]; w.N = lay.dims[l]; w.B = lay.batch; w.groups = lay.m;
    w.lr = h->lr; w.mu = h->mu;
    {
      ProfScope ps(h, LS_K_DW, l);
      LS_CUDA(h, launch_dw(w, bf, h->stream, &h->launches));
    }
    }
    if (lay.has_bias && !bias_done[l]) {
      BiasArgs b;
      b.dZ = dZ;
      b.bias = params_of(h) + lay.b_off[l];
      b.vbias = mom_of(h) + lay.b_off[l];
      b.gstride = lay.stride;
      b.B = lay.batch; b.N = lay.dims[l + 1]; b.groups = lay.m;
      b.lr = h->lr; b.mu = h->mu;
      ProfScope ps(h, LS_K_BIAS, l);
      LS_CUDA(h, launch_bias(b, bf, h->stream, &h->launches));
    }
  }
  // largest layer first, so that the short tiles fill the end of the list
  std::sort(upd, upd + n_upd, [](const TcUpdateArgs& x, const TcUpdateArgs& y) {
    return (int64_t)x.M * x.N > (int64_t)y.M * y.N;
  });
  // A step that ends in an averaging step (the last of a communication period): the streamed layers' update and
  // their average are one launch that never writes the per-replica values (and, at a period of 1, reads the old
  // state once, from the synchronized copy: upd[].mapWsync is set then); the small tensors (biases, a narrow
  // output layer), updated per replica above, are averaged by the plain kernel.
  bool fused = avg_after && n_upd > 0 && bf && h->shard_G == 0 &&
               (h->mu == 0.f ? h->spec.momentum_mode != LS_MOMENTUM_BLOCK : h->spec.momentum_mode == LS_MOMENTUM_AVERAGE);
  for (int i = 0; i < n_upd && fused; ++i) fused = tc_sync_step_shape_ok(false, upd[i].M, upd[i].N, upd[i].B);
  if (fused) {
    for (int i = 0; i < n_upd; i += tc_update_max_layers()) {
      const int n = std::min(n_upd - i, tc_update_max_layers());
      ProfScope ps(h, LS_K_AVG, 1);
      LS_CUDA(h, launch_tc_sync_step(upd + i, n, h->stream, &h->launches));
    }
    // what is left of a replica vector: the gaps between the streamed weight matrices, in layout order
    std::sort(upd, upd + n_upd, [&](const TcUpdateArgs& x, const TcUpdateArgs& y) {
      return lay.w_off[x.layer] < lay.w_off[y.layer];
    });
    const int64_t buf_stride = (int64_t)((lay.mom_off - lay.params_off) / 4);
    const int n_buf = h->mu != 0.f ? 2 : 1;
    int64_t pos = 0, begin[LS_MAX_LAYERS + 1], len[LS_MAX_LAYERS + 1];
    int n_pieces = 0;
    for (int i = 0; i <= n_upd; ++i) {
      const int64_t end = i < n_upd ? lay.w_off[upd[i].layer] : lay.stride;
      if (end > pos) { begin[n_pieces] = pos; len[n_pieces] = end - pos; ++n_pieces; }
      if (i < n_upd) pos = round_up(lay.w_off[upd[i].layer] + (int64_t)upd[i].M * upd[i].N, kAlignFloats);
    }
    {
      ProfScope ps(h, LS_K_AVG, 0);
      LS_CUDA(h, launch_average_pieces(params_of(h), n_buf, buf_stride, lay.m, begin, len, n_pieces, lay.stride, shadow_of(h),
                                       h->stream, &h->launches, sync_of(h), lay.stride));
    }
    h->sync_valid = true;
    return LS_OK;
  }
  for (int i = 0; i < n_upd; i += tc_update_max_layers()) {
    const int n = std::min(n_upd - i, tc_update_max_layers());
    ProfScope ps(h, LS_K_DW, upd[i].layer);
    LS_CUDA(h, launch_tc_update(upd + i, n, h->stream, &h->launches));
  }
  h->sync_valid = false;           // the replicas have moved apart
  if (avg_after) return average(h);
  return LS_OK;
}

static int average(ls_handle* h) {
  const Layout& lay = h->lay;
  const int64_t buf_stride = (int64_t)((lay.mom_off - lay.params_off) / 4);
  const bool both = h->mu != 0.f && h->spec.momentum_mode == LS_MOMENTUM_AVERAGE;
  const bool block = h->spec.momentum_mode == LS_MOMENTUM_BLOCK;
  if (h->shard_G >= 1) {
    // Replicas spread over G GPUs: local partial sums, one exchange, then the sum over the ranks in rank
    // order and one division by the job's replica count (see shard_average.cu).
    const int n_buf = both ? 2 : 1;
    ProfScope ps(h, LS_K_AVG, 0);
    LS_CUDA(h, launch_partial_sum(params_of(h), n_buf, buf_stride, lay.m, lay.stride, lay.stride, h->shard_partial,
                                  lay.stride, h->stream, &h->launches));
    const float* parts = h->shard_partial;
    if (h->shard_fn != nullptr) {
      const int rc = h->shard_fn(h->shard_ctx, h->shard_partial, h->shard_gathered, (size_t)n_buf * lay.stride * 4,
                                 h->shard_G);
      if (rc != 0) return LS_ERR_EXCHANGE;
      parts = h->shard_gathered;
    }
    LS_CUDA(h, launch_combine(parts, h->shard_fn ? h->shard_G : 1, (int64_t)n_buf * lay.stride, lay.stride,
                              h->shard_m_total, lay.stride, params_of(h), n_buf, buf_stride, lay.m, lay.stride,
                              shadow_of(h), h->stream, &h->launches, &h->tiles));
    if (h->mu != 0.f && h->spec.momentum_mode == LS_MOMENTUM_RESET)
      LS_CUDA(h, cudaMemsetAsync(mom_of(h), 0, (size_t)lay.m * lay.stride * 4, h->stream));
    h->sync_valid = false;         // the combining kernel keeps no synchronized copy
    return LS_OK;
  }
  {
    ProfScope ps(h, LS_K_AVG, 0);
    BlockMomentum bm{anchor_of(h), blocku_of(h), h->lr, h->spec.block_momentum};
    LS_CUDA(h, launch_average(params_of(h), both ? 2 : 1, buf_stride, lay.m, lay.stride, lay.stride,
                              shadow_of(h), h->stream, &h->launches, block ? &bm : nullptr, sync_of(h), 0, &h->tiles));
  }
  if (h->mu != 0.f && (h->spec.momentum_mode == LS_MOMENTUM_RESET || block)) {
    LS_CUDA(h, cudaMemsetAsync(mom_of(h), 0, (size_t)lay.m * lay.stride * 4, h->stream));
    LS_CUDA(h, cudaMemsetAsync(sync_of(h) + lay.stride, 0, (size_t)lay.stride * 4, h->stream));
  }
  // the synchronized copy now equals every replica: parameters always; momentum when it was averaged or
  // cleared (or is not used at all)
  h->sync_valid = h->mu == 0.f || h->spec.momentum_mode != LS_MOMENTUM_KEEP;
  return LS_OK;
}

static int eval_loss(ls_handle* h, int replica, int64_t row_offset, int64_t n_rows, float* F_host) {
  const Layout& lay = h->lay;
  if (h->x_dev == nullptr) return LS_ERR_NO_DATASET;
  if (replica < 0 || replica >= lay.m || F_host == nullptr || n_rows < lay.batch || n_rows % lay.batch != 0)
    return LS_ERR_INVALID_ARG;
  if (row_offset < 0 || row_offset + n_rows > h->n_rows) return LS_ERR_ROW_RANGE;
  const int64_t chunks = n_rows / lay.batch;
  if (chunks > kEvalCap) return LS_ERR_INVALID_ARG;
  std::vector<int64_t> offs((size_t)chunks);
  for (int64_t c = 0; c < chunks; ++c) offs[(size_t)c] = row_offset + c * lay.batch;
  int64_t* off_dev = reinterpret_cast<int64_t*>(h->state + lay.evaloff_off);
  float* loss_dev = reinterpret_cast<float*>(h->state + lay.evalloss_off);
  LS_CUDA(h, cudaMemcpyAsync(off_dev, offs.data(), (size_t)chunks * 8, cudaMemcpyHostToDevice, h->stream));
  // a wave holds as many chunks as the workspace has room for: m per wave in general (activation
  // buffers), LS_MAX_REPLICAS for a one-layer model, which needs only per-row losses and counters
  const int cap = (lay.L == 1 && head_shape_ok(lay.batch, lay.dims[1])) ? LS_MAX_REPLICAS : lay.m;
  for (int64_t c0 = 0; c0 < chunks; c0 += cap) {
    const int groups = (int)((chunks - c0 < cap) ? chunks - c0 : cap);
    int rc = forward(h, h->x_dev, XMaps{&h->maps.x_data, &h->maps_mn.x_data, &h->maps_upd.x_data}, h->y_dev, off_dev + c0, groups, replica, 0,
                     false, loss_dev + c0);
    if (rc != LS_OK) return rc;
  }
  LS_CUDA(h, cudaMemcpyAsync(h->pinned, loss_dev, (size_t)chunks * 4, cudaMemcpyDeviceToHost, h->stream));
  int* flag_host = reinterpret_cast<int*>(h->pinned + kEvalCap);
  LS_CUDA(h, cudaMemcpyAsync(flag_host, err_flag_of(h), sizeof(int), cudaMemcpyDeviceToHost, h->stream));
  LS_CUDA(h, cudaStreamSynchronize(h->stream));
  if (int rc = take_device_flag(h, *flag_host)) return rc;      // a wait ran out: the losses are not valid
  double s = 0.0;
  for (int64_t c = 0; c < chunks; ++c) s += (double)h->pinned[c];
  *F_host = (float)(s / (double)chunks);
  return LS_OK;
}

static int local_steps(ls_handle* h, int tau, const int64_t* row_offset_host, float* loss_dev, bool avg_after = false) {
  const Layout& lay = h->lay;
  if (tau < 1 || row_offset_host == nullptr) return LS_ERR_INVALID_ARG;
  if (h->x_dev == nullptr) return LS_ERR_NO_DATASET;
  for (int64_t i = 0; i < (int64_t)tau * lay.m; ++i)
    if (row_offset_host[i] < 0 || row_offset_host[i] + lay.batch > h->n_rows) return LS_ERR_ROW_RANGE;
  int64_t* off_dev = reinterpret_cast<int64_t*>(h->state + lay.rowoff_off);
  // a one-layer fp32 model that fits a CTA's shared memory: all steps of the call in one launch per chunk of
  // offsets, one CTA per replica (the per-step launches of such a model are launch-latency bound)
  const bool one_launch = lay.L == 1 && !lay.bf16 && lay.dims[0] % 4 == 0 &&
                          linear_period_ok(lay.batch, lay.dims[0], lay.dims[1], h->mu != 0.f) &&
                          reinterpret_cast<uintptr_t>(h->x_dev) % 16 == 0;
  for (int s0 = 0; s0 < tau; s0 += kRowOffCap) {
    const int n = (tau - s0 < kRowOffCap) ? tau - s0 : kRowOffCap;
    LS_CUDA(h, cudaMemcpyAsync(off_dev, row_offset_host + (int64_t)s0 * lay.m, (size_t)n * lay.m * 8,
                               cudaMemcpyHostToDevice, h->stream));
    if (one_launch) {
      {
        ProfScope ps(h, LS_K_DW, 0);
        LS_CUDA(h, launch_linear_period(static_cast<const float*>(h->x_dev), h->y_dev, off_dev,
                                        params_of(h) + lay.w_off[0], mom_of(h) + lay.w_off[0],
                                        lay.has_bias ? params_of(h) + lay.b_off[0] : nullptr, mom_of(h) + lay.b_off[0],
                                        lay.stride, loss_dev ? loss_dev + (int64_t)s0 * lay.m : nullptr, n, lay.m,
                                        lay.batch, lay.dims[0], lay.dims[1], h->spec.loss, h->lr, h->mu, h->stream,
                                        &h->launches));
      }
      h->sync_valid = false;
      if (avg_after && s0 + n == tau) {
        int rc = average(h);
        if (rc != LS_OK) return rc;
      }
      continue;
    }
    for (int s = 0; s < n; ++s) {
      const TcMaps& mnm = lay.bf16 ? h->maps : h->maps_mn;
      int rc = local_step(h, h->x_dev, XMaps{&h->maps.x_data, &mnm.x_data, &h->maps_upd.x_data}, h->y_dev, off_dev + (int64_t)s * lay.m,
                          loss_dev ? loss_dev + (int64_t)(s0 + s) * lay.m : nullptr, avg_after && s0 + s == tau - 1);
      if (rc != LS_OK) return rc;
    }
  }
  return LS_OK;
}

}  // namespace ls

// ---------------------------------------------------------------------------
// C ABI
// ---------------------------------------------------------------------------

extern "C" {

const char* ls_strerror(int code) {
  switch (code) {
    case LS_OK: return "ok";
    case LS_ERR_INVALID_ARG: return "invalid argument";
    case LS_ERR_BAD_HANDLE: return "bad handle";
    case LS_ERR_STATE_SIZE: return "state block too small or misaligned";
    case LS_ERR_NO_DATASET: return "no dataset bound";
    case LS_ERR_ROW_RANGE: return "mini-batch rows outside the dataset";
    case LS_ERR_CUDA: return "CUDA error";
    case LS_ERR_UNSUPPORTED: return "not supported";
    case LS_ERR_OVERFLOW: return "result does not fit";
    case LS_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel ran out";
    case LS_ERR_TOO_LARGE: return "size beyond the fixed capacity of this entry point";
    case LS_ERR_EXCHANGE: return "the caller's exchange of partial sums failed";
    default: return "unknown error";
  }
}

int ls_param_count(const ls_model_spec* spec, int64_t* P) {
  int rc = check_spec(spec);
  if (rc != LS_OK) return rc;
  if (P == nullptr) return LS_ERR_INVALID_ARG;
  int64_t n = 0;
  for (int l = 0; l < spec->n_layers; ++l)
    n += (int64_t)spec->dims[l + 1] * spec->dims[l] + (spec->has_bias ? spec->dims[l + 1] : 0);
  *P = n;
  return LS_OK;
}

int ls_state_bytes(int m, const ls_model_spec* spec, int batch, size_t* bytes) {
  if (bytes == nullptr) return LS_ERR_INVALID_ARG;
  Layout lay;
  int rc = make_layout(m, spec, batch, &lay);
  if (rc != LS_OK) return rc;
  *bytes = lay.total;
  return LS_OK;
}

int ls_create(ls_handle** out, int m, const ls_model_spec* spec, float lr, float momentum, int batch, void* state_dev,
              size_t state_bytes, void* cuda_stream) {
  if (out == nullptr) return LS_ERR_INVALID_ARG;
  *out = nullptr;
  Layout lay;
  int rc = make_layout(m, spec, batch, &lay);
  if (rc != LS_OK) return rc;
  if (!isfinite(lr) || !isfinite(momentum) || momentum < 0.f || momentum >= 1.f) return LS_ERR_INVALID_ARG;
  if (state_dev == nullptr || reinterpret_cast<uintptr_t>(state_dev) % 256 != 0 || state_bytes < lay.total)
    return LS_ERR_STATE_SIZE;
  ls_handle* h = new (std::nothrow) ls_handle();
  if (h == nullptr) return LS_ERR_INVALID_ARG;
  memset(h, 0, sizeof(*h));
  h->magic = kMagic;
  h->lay = lay;
  h->spec = *spec;
  h->lr = lr;
  h->mu = momentum;
  h->state = static_cast<char*>(state_dev);
  h->stream = static_cast<cudaStream_t>(cuda_stream);
  h->allow_pair = pair_kernels_enabled();
  h->allow_head_step = head_step_enabled();
  for (int l = 0; l < lay.L; ++l)
    if (lay.tiled[l]) {
      TileMap& tm = h->tiles;
      tm.begin[tm.n] = lay.w_off[l]; tm.size[tm.n] = (int64_t)lay.dims[l + 1] * lay.dims[l]; tm.cols[tm.n] = lay.dims[l];
      tm.panel[tm.n] = lay.panel[l];
      ++tm.n;
    }
  int e = cudaStreamCreateWithFlags(&h->copy_stream, cudaStreamNonBlocking);
  for (int s = 0; s < 2 && e == cudaSuccess; ++s) {
    e = cudaEventCreateWithFlags(&h->ev_copied[s], cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_consumed[s], cudaEventDisableTiming);
  }
  if (e == cudaSuccess) e = cudaMallocHost(reinterpret_cast<void**>(&h->pinned), (size_t)(kEvalCap + 16) * 4);
  // parameters, momentum, workspace start at zero; the staging row offsets are g*batch
  if (e == cudaSuccess) e = cudaMemsetAsync(h->state, 0, lay.total, h->stream);
  if (e == cudaSuccess) {
    // A tensor gets a TMA descriptor when its rows are 16-byte multiples; the tensor-core kernels are
    // only chosen for shapes (multiples of 32 / 64) whose tensors all satisfy this.
    const bool f = !lay.bf16;
    const int q = f ? 4 : 8;                       // elements per 16 bytes
    const int64_t rows = (int64_t)m * batch;
    auto ok = [&](int e2) { if (e == cudaSuccess) e = e2; };
    for (int v = 0; v < (f ? 2 : 1); ++v) {        // v = 1: the MN-major descriptors of an fp32 model
      TcMaps& mp = v ? h->maps_mn : h->maps;
      const bool mn = v != 0;
      for (int l = 0; l < lay.L; ++l) {
        if (lay.dims[l] % q == 0) {
          const void* wsrc = f ? (const void*)(params_of(h) + lay.w_off[l]) : (const void*)(shadow_of(h) + lay.w_off[l]);
          if (lay.panel[l]) ok(tc_make_panel_map(&mp.w[l], wsrc, lay.dims[l + 1], lay.dims[l], m, lay.stride));
          else ok(tc_make_map_3d(&mp.w[l], wsrc, f, mn, lay.dims[l + 1], lay.dims[l], m, lay.stride));
          if (l >= 1) {
            ok(tc_make_map_2d(&mp.act[l], h->state + lay.act_off[l], f, mn, rows, lay.dims[l]));
          }
        }
        if (lay.dims[l + 1] % q == 0) {
          ok(tc_make_map_2d(&mp.dz[l], h->state + lay.dz_off[l], f, mn, rows, lay.dims[l + 1]));
        }
      }
      if (!mn) {
        for (int l = 0; l < lay.L; ++l)
          if (lay.dims[l] % 4 == 0) {
            const bool blk = lay.tiled[l] != 0;
            ok(tc_make_block_map_3d(&mp.wf[l], params_of(h) + lay.w_off[l], lay.dims[l + 1], lay.dims[l], m, lay.stride, blk));
            ok(tc_make_block_map_3d(&mp.vf[l], mom_of(h) + lay.w_off[l], lay.dims[l + 1], lay.dims[l], m, lay.stride, blk));
            ok(tc_make_block_map_3d(&mp.wsync[l], sync_of(h) + lay.w_off[l], lay.dims[l + 1], lay.dims[l], 1, lay.stride,
                                    blk));
            ok(tc_make_block_map_3d(&mp.vsync[l], sync_of(h) + lay.stride + lay.w_off[l], lay.dims[l + 1], lay.dims[l], 1,
                                    lay.stride, blk));
          }
      }
      if (lay.dims[0] % q == 0) {
        for (int s = 0; s < 2; ++s)
          ok(tc_make_map_2d(&mp.x_stage[s], h->state + lay.stage_x_off[s], f, mn, rows, lay.dims[0]));
      }
    }
    // the operands of the update kernel: dZ_l and the layer inputs, MN-major, boxes of its stage height
    const int ur = tc_update_box_rows(f);
    for (int l = 0; l < lay.L; ++l) {
      if (l >= 1 && lay.dims[l] % q == 0)
        ok(tc_make_map_2d_rows(&h->maps_upd.act[l], h->state + lay.act_off[l], f, f, rows, lay.dims[l], ur));
      if (lay.dims[l + 1] % q == 0)
        ok(tc_make_map_2d_rows(&h->maps_upd.dz[l], h->state + lay.dz_off[l], f, f, rows, lay.dims[l + 1], ur));
    }
    if (lay.dims[0] % q == 0)
      for (int s = 0; s < 2; ++s)
        ok(tc_make_map_2d_rows(&h->maps_upd.x_stage[s], h->state + lay.stage_x_off[s], f, f, rows, lay.dims[0], ur));
  }
  if (e != cudaSuccess) {
    h->last_cuda = e;
    ls_destroy(h);
    return LS_ERR_CUDA;
  }
  *out = h;
  return LS_OK;
}

int ls_destroy(ls_handle* h) {
  if (!ok_handle(h)) return LS_ERR_BAD_HANDLE;
  cudaStreamSynchronize(h->stream);
  if (h->copy_stream) { cudaStreamSynchronize(h->copy_stream); cudaStreamDestroy(h->copy_stream); }
  for (int s = 0; s < 2; ++s) {
    if (h->ev_copied[s]) cudaEventDestroy(h->ev_copied[s]);
    if (h->ev_consumed[s]) cudaEventDestroy(h->ev_consumed[s]);
  }
  if (h->pinned) cudaFreeHost(h->pinned);
  if (h->prof_ev) {
    for (int i = 0; i < 2 * h->prof_cap; ++i) cudaEventDestroy(h->prof_ev[i]);
    delete[] h->prof_ev;
    delete[] h->prof_tag;
  }
  h->magic = 0;
  delete h;
  return LS_OK;
}

int ls_sync(ls_handle* h) {
  if (!ok_handle(h)) return LS_ERR_BAD_HANDLE;
  LS_CUDA(h, cudaStreamSynchronize(h->stream));
  LS_CUDA(h, cudaGetLastError());
  return check_device_flag(h);
}

int ls_last_cuda_error(const ls_handle* h) { return ok_handle(h) ? h->last_cuda : LS_ERR_BAD_HANDLE; }

int ls_set_lr(ls_handle* h, float lr) {
  if (!ok_handle(h)) return LS_ERR_BAD_HANDLE;
  if (!isfinite(lr)) return LS_ERR_INVALID_ARG;
  h->lr = lr;
  return LS_OK;
}

// copy one replica between the flat interface layout (host) and the padded device layout
static int copy_replica(ls_handle* h, float* dev_base, float* host, bool to_dev) {
  const Layout& lay = h->lay;
  float* stage = reinterpret_cast<float*>(h->state + lay.retile_off);
  for (int l = 0; l < lay.L; ++l) {
    const size_t wn = (size_t)lay.dims[l + 1] * lay.dims[l] * 4, bn = (size_t)lay.dims[l + 1] * 4;
    if (lay.tiled[l]) {
      // the interface is row-major, the device keeps this matrix in 32 x 32 blocks: through the staging buffer
      if (to_dev) {
        LS_CUDA(h, cudaMemcpyAsync(stage, host + lay.w_flat[l], wn, cudaMemcpyHostToDevice, h->stream));
        LS_CUDA(h, launch_retile(dev_base + lay.w_off[l], stage, lay.dims[l + 1], lay.dims[l], true, h->stream, &h->launches));
      } else {
        LS_CUDA(h, launch_retile(stage, dev_base + lay.w_off[l], lay.dims[l + 1], lay.dims[l], false, h->stream, &h->launches));
        LS_CUDA(h, cudaMemcpyAsync(host + lay.w_flat[l], stage, wn, cudaMemcpyDeviceToHost, h->stream));
      }
      if (lay.has_bias) {
        if (to_dev)
          LS_CUDA(h, cudaMemcpyAsync(dev_base + lay.b_off[l], host + lay.b_flat[l], bn, cudaMemcpyHostToDevice, h->stream));
        else
          LS_CUDA(h, cudaMemcpyAsync(host + lay.b_flat[l], dev_base + lay.b_off[l], bn, cudaMemcpyDeviceToHost, h->stream));
      }
      continue;
    }
    if (to_dev) {
      LS_CUDA(h, cudaMemcpyAsync(dev_base + lay.w_off[l], host + lay.w_flat[l], wn, cudaMemcpyHostToDevice, h->stream));
      if (lay.has_bias)
        LS_CUDA(h, cudaMemcpyAsync(dev_base + lay.b_off[l], host + lay.b_flat[l], bn, cudaMemcpyHostToDevice, h->stream));
    } else {
      LS_CUDA(h, cudaMemcpyAsync(host + lay.w_flat[l], dev_base + lay.w_off[l], wn, cudaMemcpyDeviceToHost, h->stream));
      if (lay.has_bias)
        LS_CUDA(h, cudaMemcpyAsync(host + lay.b_flat[l], dev_base + lay.b_off[l], bn, cudaMemcpyDeviceToHost, h->stream));
    }
  }
  return LS_OK;
}

int ls_set_params(ls_handle* h, const float* x1_host) {
  if (!ok_handle(h)) return LS_ERR_BAD_HANDLE;
  if (x1_host == nullptr) return LS_ERR_INVALID_ARG;
  const Layout& lay = h->lay;
  int rc = copy_replica(h, params_of(h), const_cast<float*>(x1_host), true);
  if (rc != LS_OK) return rc;
  for (int i = 1; i < lay.m; ++i)
    LS_CUDA(h, cudaMemcpyAsync(params_of(h) + (int64_t)i * lay.stride, params_of(h), (size_t)lay.stride * 4,
                               cudaMemcpyDeviceToDevice, h->stream));
  LS_CUDA(h, cudaMemsetAsync(mom_of(h), 0, (size_t)lay.m * lay.stride * 4, h->stream));
  LS_CUDA(h, cudaMemcpyAsync(sync_of(h), params_of(h), (size_t)lay.stride * 4, cudaMemcpyDeviceToDevice, h->stream));
  LS_CUDA(h, cudaMemsetAsync(sync_of(h) + lay.stride, 0, (size_t)lay.stride * 4, h->stream));
  h->sync_valid = true;
  if (h->spec.momentum_mode == LS_MOMENTUM_BLOCK) {
    LS_CUDA(h, cudaMemcpyAsync(anchor_of(h), params_of(h), (size_t)lay.stride * 4, cudaMemcpyDeviceToDevice,
                               h->stream));
    LS_CUDA(h, cudaMemsetAsync(blocku_of(h), 0, (size_t)lay.stride * 4, h->stream));
  }
  rc = refresh_shadow(h);
  if (rc != LS_OK) return rc;
  return ls_sync(h);
}

int ls_set_block_state(ls_handle* h, const float* anchor_host, const float* u_host) {
  if (!ok_handle(h)) return LS_ERR_BAD_HANDLE;
  if (h->spec.momentum_mode != LS_MOMENTUM_BLOCK) return LS_ERR_UNSUPPORTED;
  int rc = LS_OK;
  if (anchor_host) rc = copy_replica(h, anchor_of(h), const_cast<float*>(anchor_host), true);
  if (rc == LS_OK && u_host) rc = copy_replica(h, blocku_of(h), const_cast<float*>(u_host), true);
  if (rc != LS_OK) return rc;
  return ls_sync(h);
}

int ls_get_block_state(ls_handle* h, float* anchor_host, float* u_host) {
  if (!ok_handle(h)) return LS_ERR_BAD_HANDLE;
  if (h->spec.momentum_mode != LS_MOMENTUM_BLOCK) return LS_ERR_UNSUPPORTED;
  int rc = LS_OK;
  if (anchor_host) rc = copy_replica(h, anchor_of(h), anchor_host, false);
  if (rc == LS_OK && u_host) rc = copy_replica(h, blocku_of(h), u_host, false);
  if (rc != LS_OK) return rc;
  return ls_sync(h);
}

int ls_set_state(ls_handle* h, int replica, const float* params_host, const float* momentum_host) {
  if (!ok_handle(h)) return LS_ERR_BAD_HANDLE;
  if (replica < 0 || replica >= h->lay.m) return LS_ERR_INVALID_ARG;
  int rc = LS_OK;
  h->sync_valid = false;
  if (params_host)
    rc = copy_replica(h, params_of(h) + (int64_t)replica * h->lay.stride, const_cast<float*>(params_host), true);
  if (rc == LS_OK && momentum_host)
    rc = copy_replica(h, mom_of(h) + (int64_t)replica * h->lay.stride, const_cast<float*>(momentum_host), true);
  if (rc == LS_OK && params_host) rc = refresh_shadow(h);
  if (rc != LS_OK) return rc;
  return ls_sync(h);
}

int ls_get_state(ls_handle* h, int replica, float* params_host, float* momentum_host) {
  if (!ok_handle(h)) return LS_ERR_BAD_HANDLE;
  if (replica < 0 || replica >= h->lay.m) return LS_ERR_INVALID_ARG;
  int rc = LS_OK;
  if (params_host) rc = copy_replica(h, params_of(h) + (int64_t)replica * h->lay.stride, params_host, false);
  if (rc == LS_OK && momentum_host)
    rc = copy_replica(h, mom_of(h) + (int64_t)replica * h->lay.stride, momentum_host, false);
  if (rc != LS_OK) return rc;
  return ls_sync(h);
}

int ls_state_view(ls_handle* h, float** params_dev, float** momentum_dev, int64_t* stride_floats) {
  if (!ok_handle(h)) return LS_ERR_BAD_HANDLE;
  if (params_dev) *params_dev = params_of(h);
  if (momentum_dev) *momentum_dev = mom_of(h);
  if (stride_floats) *stride_floats = h->lay.stride;
  return LS_OK;
}

int ls_bind_dataset(ls_handle* h, const void* x_dev, const void* y_dev, int64_t n_rows) {
  if (!ok_handle(h)) return LS_ERR_BAD_HANDLE;
  if (x_dev == nullptr || y_dev == nullptr || n_rows < h->lay.batch) return LS_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(x_dev) % 16 != 0 || reinterpret_cast<uintptr_t>(y_dev) % 4 != 0)
    return LS_ERR_INVALID_ARG;
  if (h->lay.dims[0] % (h->lay.bf16 ? 8 : 4) == 0) {
    LS_CUDA(h, tc_make_map_2d(&h->maps.x_data, x_dev, !h->lay.bf16, false, n_rows, h->lay.dims[0]));
    if (!h->lay.bf16) LS_CUDA(h, tc_make_map_2d(&h->maps_mn.x_data, x_dev, true, true, n_rows, h->lay.dims[0]));
    LS_CUDA(h, tc_make_map_2d_rows(&h->maps_upd.x_data, x_dev, !h->lay.bf16, !h->lay.bf16, n_rows, h->lay.dims[0],
                                   tc_update_box_rows(!h->lay.bf16)));
  }
  h->x_dev = x_dev;
  h->y_dev = y_dev;
  h->n_rows = n_rows;
  return LS_OK;
}

int ls_local_steps(ls_handle* h, int tau, const int64_t* row_offset_host, float* loss_dev) {
  if (!ok_handle(h)) return LS_ERR_BAD_HANDLE;
  return local_steps(h, tau, row_offset_host, loss_dev);
}

int ls_local_steps_avg(ls_handle* h, int tau, const int64_t* row_offset_host, float* loss_dev) {
  if (!ok_handle(h)) return LS_ERR_BAD_HANDLE;
  return local_steps(h, tau, row_offset_host, loss_dev, true);
}

int ls_local_steps_host(ls_handle* h, int tau, const void* x_host, const void* y_host, float* loss_host) {
  if (!ok_handle(h)) return LS_ERR_BAD_HANDLE;
  if (tau < 1 || x_host == nullptr || y_host == nullptr || loss_host == nullptr) return LS_ERR_INVALID_ARG;
  const Layout& lay = h->lay;
  const size_t esz = lay.bf16 ? 2 : 4;
  const size_t xb = (size_t)lay.m * lay.batch * lay.dims[0] * esz, yb = (size_t)lay.m * lay.batch * 4;
  // group g of a staged step reads rows [g*batch, +batch) of the staging buffer
  int64_t* stage_off = reinterpret_cast<int64_t*>(h->state + lay.evaloff_off);
  {
    int64_t offs[LS_MAX_REPLICAS];
    for (int g = 0; g < lay.m; ++g) offs[g] = (int64_t)g * lay.batch;
    LS_CUDA(h, cudaMemcpyAsync(stage_off, offs, (size_t)lay.m * 8, cudaMemcpyHostToDevice, h->stream));
    LS_CUDA(h, cudaStreamSynchronize(h->stream));
  }
  float* loss_stage = reinterpret_cast<float*>(h->state + lay.stage_loss_off);
  bool used[2] = {false, false};
  for (int s0 = 0; s0 < tau; s0 += kRowOffCap) {
    const int n = (tau - s0 < kRowOffCap) ? tau - s0 : kRowOffCap;
    for (int s = 0; s < n; ++s) {
      const int slot = (s0 + s) & 1;
      void* xs = h->state + lay.stage_x_off[slot];
      void* ys = h->state + lay.stage_y_off[slot];
      if (used[slot]) LS_CUDA(h, cudaStreamWaitEvent(h->copy_stream, h->ev_consumed[slot], 0));
      LS_CUDA(h, cudaMemcpyAsync(xs, static_cast<const char*>(x_host) + (size_t)(s0 + s) * xb, xb,
                                 cudaMemcpyHostToDevice, h->copy_stream));
      LS_CUDA(h, cudaMemcpyAsync(ys, static_cast<const char*>(y_host) + (size_t)(s0 + s) * yb, yb,
                                 cudaMemcpyHostToDevice, h->copy_stream));
      LS_CUDA(h, cudaEventRecord(h->ev_copied[slot], h->copy_stream));
      LS_CUDA(h, cudaStreamWaitEvent(h->stream, h->ev_copied[slot], 0));
      const TcMaps& mnm = lay.bf16 ? h->maps : h->maps_mn;
      int rc = local_step(h, xs, XMaps{&h->maps.x_stage[slot], &mnm.x_stage[slot], &h->maps_upd.x_stage[slot]}, ys,
                          stage_off,
                          loss_stage + (int64_t)s * lay.m);
      if (rc != LS_OK) return rc;
      LS_CUDA(h, cudaEventRecord(h->ev_consumed[slot], h->stream));
      used[slot] = true;
    }
    LS_CUDA(h, cudaMemcpyAsync(loss_host + (int64_t)s0 * lay.m, loss_stage, (size_t)n * lay.m * 4,
                               cudaMemcpyDeviceToHost, h->stream));
    if (int rc = check_device_flag(h)) return rc;        // waits for the stream; a wait that ran out ends the call
  }
  return LS_OK;
}

int ls_average(ls_handle* h) {
  if (!ok_handle(h)) return LS_ERR_BAD_HANDLE;
  return average(h);
}

int ls_eval_loss(ls_handle* h, int replica, int64_t row_offset, int64_t n_rows, float* F_host) {
  if (!ok_handle(h)) return LS_ERR_BAD_HANDLE;
  return eval_loss(h, replica, row_offset, n_rows, F_host);
}

int ls_shard_buffer_floats(const ls_handle* h, int64_t* floats) {
  if (!ok_handle(h)) return LS_ERR_BAD_HANDLE;
  if (floats == nullptr) return LS_ERR_INVALID_ARG;
  *floats = 2 * h->lay.stride;
  return LS_OK;
}

int ls_set_shard(ls_handle* h, int n_gpus, int m_total, float* partial_dev, float* gathered_dev, ls_exchange_fn exchange,
                 void* ctx) {
  if (!ok_handle(h)) return LS_ERR_BAD_HANDLE;
  if (n_gpus == 0) {                       // back to a job that lives on this GPU alone
    h->shard_G = 0; h->shard_fn = nullptr; h->shard_ctx = nullptr;
    return LS_OK;
  }
  if (h->spec.momentum_mode == LS_MOMENTUM_BLOCK) return LS_ERR_UNSUPPORTED;
  if (n_gpus < 1 || m_total != n_gpus * h->lay.m || partial_dev == nullptr) return LS_ERR_INVALID_ARG;
  if (n_gpus > 1 && (exchange == nullptr || gathered_dev == nullptr)) return LS_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(partial_dev) % 256 != 0 || reinterpret_cast<uintptr_t>(gathered_dev) % 256 != 0)
    return LS_ERR_INVALID_ARG;
  h->shard_G = n_gpus; h->shard_m_total = m_total;
  h->shard_partial = partial_dev; h->shard_gathered = gathered_dev;
  h->shard_fn = n_gpus > 1 ? exchange : nullptr; h->shard_ctx = ctx;
  return LS_OK;
}

int ls_shard_partial_sum(ls_handle* h, float* partial_dev) {
  if (!ok_handle(h)) return LS_ERR_BAD_HANDLE;
  if (partial_dev == nullptr || reinterpret_cast<uintptr_t>(partial_dev) % 256 != 0) return LS_ERR_INVALID_ARG;
  const Layout& lay = h->lay;
  const bool both = h->mu != 0.f && h->spec.momentum_mode == LS_MOMENTUM_AVERAGE;
  LS_CUDA(h, launch_partial_sum(params_of(h), both ? 2 : 1, (int64_t)((lay.mom_off - lay.params_off) / 4), lay.m,
                                lay.stride, lay.stride, partial_dev, lay.stride, h->stream, &h->launches));
  return LS_OK;
}

int ls_shard_average(ls_handle* h, const float* gathered_dev, int n_gpus, int m_total) {
  if (!ok_handle(h)) return LS_ERR_BAD_HANDLE;
  if (h->spec.momentum_mode == LS_MOMENTUM_BLOCK) return LS_ERR_UNSUPPORTED;
  if (gathered_dev == nullptr || reinterpret_cast<uintptr_t>(gathered_dev) % 256 != 0 || n_gpus < 1 ||
      m_total != n_gpus * h->lay.m)
    return LS_ERR_INVALID_ARG;
  const Layout& lay = h->lay;
  const bool both = h->mu != 0.f && h->spec.momentum_mode == LS_MOMENTUM_AVERAGE;
  const int n_buf = both ? 2 : 1;
  LS_CUDA(h, launch_combine(gathered_dev, n_gpus, (int64_t)n_buf * lay.stride, lay.stride, m_total, lay.stride,
                            params_of(h), n_buf, (int64_t)((lay.mom_off - lay.params_off) / 4), lay.m, lay.stride,
                            shadow_of(h), h->stream, &h->launches, &h->tiles));
  if (h->mu != 0.f && h->spec.momentum_mode == LS_MOMENTUM_RESET)
    LS_CUDA(h, cudaMemsetAsync(mom_of(h), 0, (size_t)lay.m * lay.stride * 4, h->stream));
  h->sync_valid = false;
  return LS_OK;
}

int adacomm_next_tau(double F_t, double F_0, int tau_0) {
  if (!isfinite(F_t) || !isfinite(F_0) || !(F_0 > 0.0) || F_t < 0.0 || tau_0 < 1) return LS_ERR_INVALID_ARG;
  const double ratio = F_t / F_0;
  const double t = sqrt(ratio) * (double)tau_0;
  double n = ceil(t);
  if (n < 1.0) n = 1.0;
  if (!(n <= 2147483647.0)) return LS_ERR_OVERFLOW;
  return (int)n;
}

int adacomm_next_tau_refined(double F_t, double F_0, int tau_0, int tau_prev, double gamma, int slack, double lr_0,
                             double lr_l, int lr_changed) {
  if (!isfinite(F_t) || !isfinite(F_0) || !isfinite(gamma) || !isfinite(lr_0) || !isfinite(lr_l)) return LS_ERR_INVALID_ARG;
  if (!(F_0 > 0.0) || F_t < 0.0 || tau_0 < 1 || tau_prev < 1 || !(gamma > 0.0 && gamma <= 1.0) || slack < 0 ||
      !(lr_0 > 0.0) || !(lr_l > 0.0))
    return LS_ERR_INVALID_ARG;
  const double scaled = (lr_0 / lr_l) * (F_t / F_0);
  double c = ceil(sqrt(scaled) * (double)tau_0);
  if (c < 1.0) c = 1.0;
  if (!(c <= 2147483647.0)) return LS_ERR_OVERFLOW;
  if (lr_changed || c + (double)slack < (double)tau_prev) return (int)c;
  double n = ceil(gamma * (double)tau_prev);
  if (n < 1.0) n = 1.0;
  return (int)n;
}

static int run_loop(ls_handle* h, int64_t K, int tau_0, int interval, int64_t probe_rows, const int64_t* row_offset_host,
                    float* loss_dev, int32_t* period_tau, int64_t max_periods, int64_t* n_periods, int64_t* decision_k,
                    float* decision_F, int32_t* decision_tau, int64_t max_decisions, int64_t* n_decisions,
                    float* F0_host, const ls_adacomm_opts* opts, bool timed = false, double t0_ms = 0.0,
                    double* decision_ms = nullptr);

int ls_run_timed(ls_handle* h, int64_t K, int tau_0, double T0_ms, int64_t probe_rows, const int64_t* row_offset_host,
                 float* loss_dev, int32_t* period_tau, int64_t max_periods, int64_t* n_periods, int64_t* decision_k,
                 float* decision_F, int32_t* decision_tau, double* decision_ms, int64_t max_decisions,
                 int64_t* n_decisions, float* F0_host) {
  if (!isfinite(T0_ms)) return LS_ERR_INVALID_ARG;
  return run_loop(h, K, tau_0, 1, probe_rows, row_offset_host, loss_dev, period_tau, max_periods, n_periods,
                  decision_k, decision_F, decision_tau, max_decisions, n_decisions, F0_host, nullptr, true, T0_ms,
                  decision_ms);
}

int ls_run(ls_handle* h, int64_t K, int tau_0, int interval, int64_t probe_rows, const int64_t* row_offset_host,
           float* loss_dev, int32_t* period_tau, int64_t max_periods, int64_t* n_periods, int64_t* decision_k,
           float* decision_F, int32_t* decision_tau, int64_t max_decisions, int64_t* n_decisions, float* F0_host) {
  return run_loop(h, K, tau_0, interval, probe_rows, row_offset_host, loss_dev, period_tau, max_periods, n_periods,
                  decision_k, decision_F, decision_tau, max_decisions, n_decisions, F0_host, nullptr);
}

int ls_run_refined(ls_handle* h, int64_t K, int tau_0, int interval, int64_t probe_rows,
                   const int64_t* row_offset_host, float* loss_dev, const ls_adacomm_opts* opts, int32_t* period_tau,
                   int64_t max_periods, int64_t* n_periods, int64_t* decision_k, float* decision_F,
                   int32_t* decision_tau, int64_t max_decisions, int64_t* n_decisions, float* F0_host) {
  if (opts == nullptr || interval < 1) return LS_ERR_INVALID_ARG;
  if (!isfinite(opts->gamma) || !(opts->gamma > 0.0 && opts->gamma <= 1.0) || opts->slack < 0 || opts->n_decay < 0 ||
      (opts->n_decay > 0 && (opts->decay_at == nullptr || !isfinite(opts->decay_factor) || !(opts->decay_factor > 0.0))))
    return LS_ERR_INVALID_ARG;
  for (int i = 1; i < opts->n_decay; ++i)
    if (opts->decay_at[i] < opts->decay_at[i - 1]) return LS_ERR_INVALID_ARG;
  return run_loop(h, K, tau_0, interval, probe_rows, row_offset_host, loss_dev, period_tau, max_periods, n_periods,
                  decision_k, decision_F, decision_tau, max_decisions, n_decisions, F0_host, opts);
}

}  // extern "C"

static int run_loop(ls_handle* h, int64_t K, int tau_0, int interval, int64_t probe_rows, const int64_t* row_offset_host,
                    float* loss_dev, int32_t* period_tau, int64_t max_periods, int64_t* n_periods, int64_t* decision_k,
                    float* decision_F, int32_t* decision_tau, int64_t max_decisions, int64_t* n_decisions,
                    float* F0_host, const ls_adacomm_opts* opts, bool timed, double t0_ms, double* decision_ms) {
  if (!ok_handle(h)) return LS_ERR_BAD_HANDLE;
  if (K < 1 || tau_0 < 1 || interval < 0 || row_offset_host == nullptr) return LS_ERR_INVALID_ARG;
  const Layout& lay = h->lay;
  const double lr_0 = (double)h->lr;
  int next_decay = 0;
  float F_0 = 0.f;
  if (interval > 0) {
    int rc = eval_loss(h, 0, 0, probe_rows, &F_0);
    if (rc != LS_OK) return rc;
    if (F0_host) *F0_host = F_0;
  }
  int64_t k = 0, np = 0, nd = 0, next_interval = 1;
  int tau = tau_0;
  const auto t_start = std::chrono::steady_clock::now();
  while (k < K) {
    const int steps = (int)((K - k < tau) ? K - k : tau);
    if (period_tau && np < max_periods) period_tau[np] = tau;
    ++np;
    // the period's local steps, then its averaging step
    int rc = local_steps(h, steps, row_offset_host + k * lay.m, loss_dev ? loss_dev + k * lay.m : nullptr, true);
    if (rc != LS_OK) return rc;
    k += steps;
    bool decide = interval > 0 && k >= next_interval * (int64_t)interval;
    double elapsed_ms = 0.0;
    if (timed) {
      // wall-clock intervals (Section 4): the averaging step has to be over before the clock is read
      if (int frc = check_device_flag(h)) return frc;      // waits for the stream
      elapsed_ms = std::chrono::duration<double, std::milli>(std::chrono::steady_clock::now() - t_start).count();
      decide = t0_ms <= 0.0 || elapsed_ms >= (double)next_interval * t0_ms;
    }
    if (decide) {
      float F_t = 0.f;
      rc = eval_loss(h, 0, 0, probe_rows, &F_t);
      if (rc != LS_OK) return rc;
      int t;
      if (opts != nullptr) {
        // Section 4.3: a scheduled learning-rate decay waits until the period in force is 1
        int changed = 0;
        if (next_decay < opts->n_decay && opts->decay_at[next_decay] <= k && tau == 1) {
          ++next_decay;
          h->lr = (float)((double)h->lr * opts->decay_factor);
          changed = 1;
        }
        t = adacomm_next_tau_refined((double)F_t, (double)F_0, tau_0, tau, opts->gamma, opts->slack, lr_0, (double)h->lr,
                                     changed);
      } else {
        t = adacomm_next_tau((double)F_t, (double)F_0, tau_0);
      }
      if (t < 0) return t;
      tau = t;
      if (nd < max_decisions) {
        if (decision_k) decision_k[nd] = k;
        if (decision_F) decision_F[nd] = F_t;
        if (decision_tau) decision_tau[nd] = t;
        if (decision_ms) decision_ms[nd] = elapsed_ms;
      }
      ++nd;
      if (timed) next_interval = t0_ms > 0.0 ? (int64_t)floor(elapsed_ms / t0_ms) + 1 : 1;
      else next_interval = k / interval + 1;
    }
  }
  if (n_periods) *n_periods = np;
  if (n_decisions) *n_decisions = nd;
  return LS_OK;
}

extern "C" {

int ls_selftest_wait_timeout(ls_handle* h, int64_t limit_cycles) {
  if (!ok_handle(h)) return LS_ERR_BAD_HANDLE;
  if (limit_cycles < 1 || limit_cycles > 2000000000ll) return LS_ERR_INVALID_ARG;
  wait_timeout_selftest_kernel<<<1, 32, 0, h->stream>>>(err_flag_of(h), (long long)limit_cycles);
  ++h->launches;
  LS_CUDA(h, cudaGetLastError());
  return LS_OK;
}

int ls_get_lr(const ls_handle* h, float* lr) {
  if (!ok_handle(h)) return LS_ERR_BAD_HANDLE;
  if (lr == nullptr) return LS_ERR_INVALID_ARG;
  *lr = h->lr;
  return LS_OK;
}

int ls_profile_begin(ls_handle* h, uint32_t class_mask, int layer) {
  if (!ok_handle(h)) return LS_ERR_BAD_HANDLE;
  if (layer >= LS_MAX_LAYERS || class_mask >= (1u << LS_K_CLASSES)) return LS_ERR_INVALID_ARG;
  if (h->prof_ev == nullptr) {
    h->prof_ev = new (std::nothrow) cudaEvent_t[2 * kProfCap];
    h->prof_tag = new (std::nothrow) int16_t[kProfCap];
    if (h->prof_ev == nullptr || h->prof_tag == nullptr) return LS_ERR_INVALID_ARG;
    h->prof_cap = 0;
    for (int i = 0; i < 2 * kProfCap; ++i) {
      LS_CUDA(h, cudaEventCreate(&h->prof_ev[i]));
      if (i & 1) h->prof_cap = (i + 1) / 2;
    }
  }
  h->prof_used = 0;
  h->prof_layer = layer;
  h->prof_mask = class_mask;
  return LS_OK;
}

int ls_profile_end(ls_handle* h, double* ms, int64_t* launches) {
  if (!ok_handle(h)) return LS_ERR_BAD_HANDLE;
  if (ms == nullptr || launches == nullptr) return LS_ERR_INVALID_ARG;
  h->prof_mask = 0;
  LS_CUDA(h, cudaStreamSynchronize(h->stream));
  for (int i = 0; i < LS_K_CLASSES * LS_MAX_LAYERS; ++i) { ms[i] = 0.0; launches[i] = 0; }
  for (int r = 0; r < h->prof_used; ++r) {
    float t = 0.f;
    LS_CUDA(h, cudaEventElapsedTime(&t, h->prof_ev[2 * r], h->prof_ev[2 * r + 1]));
    ms[h->prof_tag[r]] += (double)t;
    launches[h->prof_tag[r]] += 1;
  }
  h->prof_used = 0;
  return LS_OK;
}

int ls_launch_count(const ls_handle* h, int64_t* n) {
  if (!ok_handle(h)) return LS_ERR_BAD_HANDLE;
  if (n == nullptr) return LS_ERR_INVALID_ARG;
  *n = h->launches;
  return LS_OK;
}

}  // extern "C"
