// The narrow output layer of a TRAINING step in one launch, for wide bf16 inputs (the last hidden layer of an
// MLP with thousands of units): product, per-sample loss, both gradients and the SGD-momentum update
// (Section 2 mini-batch SGD update, Section 5.3 momentum), which head_fwd_wide_kernel + head_bwd_kernel do in
// two launches and two passes over the layer input.
//
// The B rows of a replica's mini-batch are cut into 8 blocks; a CTA keeps one block of the layer input A (at most
// 32 rows x K bf16) and the whole C x K weight matrix in shared memory for the whole kernel.  Four CTAs form a
// thread-block cluster (one half of the rows), two clusters share a replica:
//
//   1. forward     z = A W^T + b for the CTA's rows: warp = 4 rows x half of K, a lane takes 4 of every 128
//                  columns; lanes are combined by a butterfly whose first two levels halve the data.
//   2. loss        one lane per row: softmax cross-entropy, dZ = (softmax - onehot) / B.
//   3. backward    a thread owns 4 columns: dPrev = (dZ W) * 1[A > 0] goes to global memory row by row, and the
//                  thread's share of G = dZ^T A (the CTA's rows only) replaces the weights it has read, in place;
//                  the column sums of dPrev (bias gradient of the layer below) are kept beside it.
//   4. exchange    cluster barrier; CTA r adds the 4 partial G of columns [r K/4, (r+1) K/4) in rank order through
//                  distributed shared memory and leaves the sum in global memory; of the two CTAs that hold the
//                  same columns (one per cluster), the one that arrives second (a counter, no waiting) adds the
//                  two sums and finishes v <- mu v + G, W <- W - eta v (and the bf16 copy); the same for the bias
//                  of the layer below, this layer's bias and the mean loss.
//
// (One cluster of 8 per replica would need no global step, but only 15 such clusters are resident at a time on
// this GPU with one CTA per SM: the 16 replicas of the large workload took two rounds, 51 us instead of 29.)
// Every sum runs in a fixed order (rows ascending inside a CTA, CTAs in rank order, half 0 + half 1), so a step is
// reproducible.  W is read from the fp32 master copy, like the two-kernel path.
#include "ls_internal.h"
#include "tc_ptx.cuh"

namespace ls {
namespace {
using namespace ptx;

constexpr int kStepThreads = 512;
constexpr int kStepCluster = 4;         // CTAs per cluster
constexpr int kStepBlocks = 8;          // row blocks per replica = 2 clusters
constexpr int kStepMaxRows = 32;        // rows per CTA
constexpr int kStepOwn4 = 3;            // 4-column groups of the owned C x K/4 block per thread, at most
constexpr int kDzLd = 12;               // floats per row of dZ / logits in shared memory (16-byte rows)

__device__ __forceinline__ float4 add4(float4 a, float4 b) { return make_float4(a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w); }
__device__ __forceinline__ float4 ld_cluster_f32x4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ void bf16x4_to_f(uint2 u, float (&r)[4]) {
  r[0] = __uint_as_float(u.x << 16); r[1] = __uint_as_float(u.x & 0xFFFF0000u);
  r[2] = __uint_as_float(u.y << 16); r[3] = __uint_as_float(u.y & 0xFFFF0000u);
}

struct StepLayout {
  size_t w, cs, slab, zpart, dz, small, total;
};
__host__ __device__ inline StepLayout step_layout(int CT, int K, int rpc) {
  StepLayout l;
  size_t o = 0;
  l.w = o; o += (size_t)CT * K * 4;            // [CT][K] fp32: W, then this CTA's partial G
  l.cs = o; o += (size_t)K * 4;                // [K] partial column sums of dPrev
  l.slab = o; o += (size_t)rpc * K * 2;        // [rpc][K] bf16: the CTA's rows of A
  l.zpart = o; o += 2 * kStepMaxRows * kDzLd * 4;
  l.dz = o; o += kStepMaxRows * kDzLd * 4;
  l.small = o; o += 32 * 4;                    // [0]: partial loss sum, [1 + c]: partial column sums of dZ
  l.total = o;
  return l;
}

template <int CT>
__global__ void __launch_bounds__(kStepThreads, 1)
head_step_kernel(const __nv_bfloat16* __restrict__ A, const int32_t* __restrict__ y,
                 const int64_t* __restrict__ y_row_off, float* __restrict__ W, float* __restrict__ V,
                 __nv_bfloat16* __restrict__ Wb, float* __restrict__ bias, float* __restrict__ vbias, int64_t w_gstride,
                 __nv_bfloat16* __restrict__ dPrev, float* __restrict__ pbias, float* __restrict__ pvbias,
                 float* __restrict__ loss_out, float* __restrict__ scratch, int64_t scratch_stride,
                 unsigned int* __restrict__ counters, int B, int K, float lr, float mu) {
  extern __shared__ __align__(16) uint8_t smem[];
  __shared__ unsigned int is_last;
  const int rpc = B / kStepBlocks;
  const StepLayout lo = step_layout(CT, K, rpc);
  float* wbuf = reinterpret_cast<float*>(smem + lo.w);
  float* cs = reinterpret_cast<float*>(smem + lo.cs);
  const __nv_bfloat16* slab = reinterpret_cast<const __nv_bfloat16*>(smem + lo.slab);
  float* zpart = reinterpret_cast<float*>(smem + lo.zpart);
  float* dz = reinterpret_cast<float*>(smem + lo.dz);
  float* small = reinterpret_cast<float*>(smem + lo.small);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int r = (int)cluster_ctarank();
  const int half = blockIdx.y, g = blockIdx.z;
  const int row0 = (half * kStepCluster + r) * rpc;        // first row of this CTA inside the replica
  const int KO = K / kStepCluster;                         // columns whose update this CTA finishes
  float* Wg = W + (int64_t)g * w_gstride;
  float* Vg = V + (int64_t)g * w_gstride;
  const float invB = 1.0f / (float)B;

  grid_dep_wait();
  grid_dep_launch();

  // ---- requests: W and the CTA's rows of A (asynchronous copies), labels and bias ---------------------------
  {
    const uint32_t wdst = smem_u32(wbuf), sdst = smem_u32(slab);
    const char* wsrc = reinterpret_cast<const char*>(Wg);
    const char* ssrc = reinterpret_cast<const char*>(A + ((int64_t)g * B + row0) * K);
    for (int i = tid; i < CT * K / 4; i += kStepThreads)
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(wdst + i * 16), "l"(wsrc + (int64_t)i * 16) : "memory");
    for (int i = tid; i < rpc * K / 8; i += kStepThreads)
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(sdst + i * 16), "l"(ssrc + (int64_t)i * 16) : "memory");
    asm volatile("cp.async.commit_group;" ::: "memory");
  }
  int label = -1;
  float bz[CT];
#pragma unroll
  for (int c = 0; c < CT; ++c) bz[c] = 0.f;
  if (warp == 0) {
    if (lane < rpc) label = y[y_row_off[g] + row0 + lane];
    if (bias != nullptr) {
#pragma unroll
      for (int c = 0; c < CT; ++c) bz[c] = bias[(int64_t)g * w_gstride + c];
    }
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  __syncthreads();

  // ---- 1. forward: warp = rows [4 (warp & 7), + 4) x slices of half (warp >> 3) of K --------------------------
  {
    const int rbase = (warp & 7) * 4, kh = warp >> 3;
    const int slices = K / 128, per = (slices + 1) / 2;
    const int s_begin = kh * per, s_end = min(slices, s_begin + per);
    if (rbase < rpc) {
      float acc[4 * CT];
#pragma unroll
      for (int i = 0; i < 4 * CT; ++i) acc[i] = 0.f;
      for (int s = s_begin; s < s_end; ++s) {
        const int k = s * 128 + lane * 4;
        float a[4][4];
#pragma unroll
        for (int rr = 0; rr < 4; ++rr)
          bf16x4_to_f(*reinterpret_cast<const uint2*>(slab + (size_t)(rbase + rr) * K + k), a[rr]);
#pragma unroll
        for (int c = 0; c < CT; ++c) {
          const float4 w = *reinterpret_cast<const float4*>(wbuf + (size_t)c * K + k);
#pragma unroll
          for (int rr = 0; rr < 4; ++rr)
            acc[rr * CT + c] = fmaf(a[rr][3], w.w, fmaf(a[rr][2], w.z, fmaf(a[rr][1], w.y, fmaf(a[rr][0], w.x, acc[rr * CT + c]))));
        }
      }
      // lane sums.  Level 1 (lane ^ 16): each side keeps rows {0, 1} or {2, 3}; level 2 (lane ^ 8): one row;
      // then a plain butterfly over the 8 lanes that hold the same row.
      const bool up1 = (lane & 16) != 0, up2 = (lane & 8) != 0;
      float u[2 * CT];
#pragma unroll
      for (int i = 0; i < 2 * CT; ++i) {
        const float keep = up1 ? acc[2 * CT + i] : acc[i];
        const float send = up1 ? acc[i] : acc[2 * CT + i];
        u[i] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
      }
      float t[CT];
#pragma unroll
      for (int i = 0; i < CT; ++i) {
        const float keep = up2 ? u[CT + i] : u[i];
        const float send = up2 ? u[i] : u[CT + i];
        t[i] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
      }
#pragma unroll
      for (int o = 4; o > 0; o >>= 1)
#pragma unroll
        for (int i = 0; i < CT; ++i) t[i] += __shfl_xor_sync(0xffffffffu, t[i], o);
      if ((lane & 7) == 0) {
        const int row = rbase + (up1 ? 2 : 0) + (up2 ? 1 : 0);
#pragma unroll
        for (int c = 0; c < CT; ++c) zpart[(kh * kStepMaxRows + row) * kDzLd + c] = t[c];
      }
    }
  }
  __syncthreads();

  // ---- 2. loss and dZ of the CTA's rows: one lane per row -------------------------------------------------------
  if (warp == 0) {
    float loss = 0.f, d[CT];
#pragma unroll
    for (int c = 0; c < CT; ++c) d[c] = 0.f;
    if (lane < rpc) {
      float z[CT], mx = -INFINITY;
#pragma unroll
      for (int c = 0; c < CT; ++c) {
        z[c] = (zpart[lane * kDzLd + c] + zpart[(kStepMaxRows + lane) * kDzLd + c]) + bz[c];
        mx = fmaxf(mx, z[c]);
      }
      float e[CT], sum = 0.f;
#pragma unroll
      for (int c = 0; c < CT; ++c) { e[c] = expf(z[c] - mx); sum += e[c]; }
      const bool valid = label >= 0 && label < CT;
      float zy = mx;
#pragma unroll
      for (int c = 0; c < CT; ++c) if (valid && c == label) zy = z[c];
      loss = (mx + logf(sum)) - zy;
#pragma unroll
      for (int c = 0; c < CT; ++c) {
        d[c] = (e[c] / sum - (c == label ? 1.f : 0.f)) * invB;
        dz[lane * kDzLd + c] = d[c];
      }
#pragma unroll
      for (int c = CT; c < kDzLd; ++c) dz[lane * kDzLd + c] = 0.f;
    }
    // this CTA's share of the loss sum and of the column sums of dZ (rows in lane order through the butterfly)
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      loss += __shfl_xor_sync(0xffffffffu, loss, o);
#pragma unroll
      for (int c = 0; c < CT; ++c) d[c] += __shfl_xor_sync(0xffffffffu, d[c], o);
    }
    if (lane == 0) {
      small[0] = loss;
#pragma unroll
      for (int c = 0; c < CT; ++c) small[1 + c] = d[c];
    }
  }
  __syncthreads();

  // ---- 3. backward: a thread owns columns [k, k + 4) ------------------------------------------------------------
  for (int k = tid * 4; k < K; k += kStepThreads * 4) {
    float w[CT][4], gw[CT][4], csum[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int c = 0; c < CT; ++c) {
      const float4 v = *reinterpret_cast<const float4*>(wbuf + (size_t)c * K + k);
      w[c][0] = v.x; w[c][1] = v.y; w[c][2] = v.z; w[c][3] = v.w;
      gw[c][0] = gw[c][1] = gw[c][2] = gw[c][3] = 0.f;
    }
    __nv_bfloat16* out = dPrev + ((int64_t)g * B + row0) * K + k;
#pragma unroll 1
    for (int row = 0; row < rpc; ++row) {
      float a[4], dr[kDzLd];
      bf16x4_to_f(*reinterpret_cast<const uint2*>(slab + (size_t)row * K + k), a);
#pragma unroll
      for (int i = 0; i < kDzLd / 4; ++i) {
        const float4 v = *reinterpret_cast<const float4*>(dz + row * kDzLd + 4 * i);
        dr[4 * i] = v.x; dr[4 * i + 1] = v.y; dr[4 * i + 2] = v.z; dr[4 * i + 3] = v.w;
      }
      float da[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int c = 0; c < CT; ++c)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          da[j] = fmaf(dr[c], w[c][j], da[j]);
          gw[c][j] = fmaf(dr[c], a[j], gw[c][j]);
        }
      float o[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        o[j] = a[j] > 0.f ? da[j] : 0.f;
        csum[j] += o[j];
      }
      __nv_bfloat162 p0 = __floats2bfloat162_rn(o[0], o[1]), p1 = __floats2bfloat162_rn(o[2], o[3]);
      *reinterpret_cast<uint2*>(out + (int64_t)row * K) =
          make_uint2(*reinterpret_cast<uint32_t*>(&p0), *reinterpret_cast<uint32_t*>(&p1));
    }
    // the partial G takes the place of the weights this thread has read (no other thread touches them)
#pragma unroll
    for (int c = 0; c < CT; ++c)
      *reinterpret_cast<float4*>(wbuf + (size_t)c * K + k) = make_float4(gw[c][0], gw[c][1], gw[c][2], gw[c][3]);
    *reinterpret_cast<float4*>(cs + k) = make_float4(csum[0], csum[1], csum[2], csum[3]);
  }

  // ---- 4. exchange ---------------------------------------------------------------------------------------------
  // Everything below moves in groups of four consecutive columns (16 bytes).  Group e = tid + i * 512 of the
  // CT x KO block this CTA owns: class e / (KO / 4), columns r KO + 4 (e mod (KO / 4)) ...
  // (the old values are requested before the barrier, so their round trip overlaps the wait)
  const int KO4 = KO / 4;
  float4 wu[kStepOwn4], vu[kStepOwn4];
#pragma unroll
  for (int i = 0; i < kStepOwn4; ++i) {
    const int e = tid + i * kStepThreads;
    wu[i] = vu[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (e < CT * KO4) {
      const int64_t at = (int64_t)(e / KO4) * K + r * KO + (e % KO4) * 4;
      wu[i] = *reinterpret_cast<const float4*>(Wg + at);
      if (mu != 0.f) vu[i] = *reinterpret_cast<const float4*>(Vg + at);
    }
  }
  float4 b_prev = make_float4(0.f, 0.f, 0.f, 0.f), vb_prev = b_prev;
  float b_own = 0.f, vb_own = 0.f;
  const bool prev_bias = pbias != nullptr && tid < KO4;
  if (prev_bias) {
    b_prev = *reinterpret_cast<const float4*>(pbias + (int64_t)g * w_gstride + r * KO + tid * 4);
    if (mu != 0.f) vb_prev = *reinterpret_cast<const float4*>(pvbias + (int64_t)g * w_gstride + r * KO + tid * 4);
  }
  if (r == 0 && bias != nullptr && tid >= 1 && tid <= CT) {       // thread 1 + c: this layer's bias c
    b_own = bias[(int64_t)g * w_gstride + tid - 1];
    if (mu != 0.f) vb_own = vbias[(int64_t)g * w_gstride + tid - 1];
  }
  cluster_sync_all();
  // 4a. inside the cluster: the owner of a column adds the 4 partial sums in rank order (distributed shared memory)
  float4 sw[kStepOwn4], sc = make_float4(0.f, 0.f, 0.f, 0.f);
  float ss = 0.f;
  {
    const uint32_t wbase = smem_u32(wbuf), cbase = smem_u32(cs), sbase = smem_u32(small);
    uint32_t peer_w[kStepCluster], peer_c[kStepCluster];
#pragma unroll
    for (int j = 0; j < kStepCluster; ++j) {
      peer_w[j] = map_to_rank(wbase, (uint32_t)j);
      peer_c[j] = map_to_rank(cbase, (uint32_t)j);
    }
#pragma unroll
    for (int i = 0; i < kStepOwn4; ++i) {
      const int e = tid + i * kStepThreads;
      sw[i] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (e < CT * KO4) {
        const uint32_t at = (uint32_t)((e / KO4) * K + r * KO + (e % KO4) * 4);
        float4 p[kStepCluster];
#pragma unroll
        for (int j = 0; j < kStepCluster; ++j) p[j] = ld_cluster_f32x4(peer_w[j] + at * 4);
        sw[i] = p[0];
#pragma unroll
        for (int j = 1; j < kStepCluster; ++j) sw[i] = add4(sw[i], p[j]);
      }
    }
    if (tid < KO4) {
      float4 p[kStepCluster];
#pragma unroll
      for (int j = 0; j < kStepCluster; ++j) p[j] = ld_cluster_f32x4(peer_c[j] + (uint32_t)((r * KO + tid * 4) * 4));
      sc = p[0];
#pragma unroll
      for (int j = 1; j < kStepCluster; ++j) sc = add4(sc, p[j]);
    }
    if (r == 0 && tid <= CT) {
      // slot 0: the loss sum; slot 1 + c: column sum of dZ (this layer's bias gradient)
#pragma unroll
      for (int j = 0; j < kStepCluster; ++j) {
        const float v = ld_cluster_f32(map_to_rank(sbase, (uint32_t)j) + (uint32_t)(tid * 4));
        ss = j == 0 ? v : ss + v;
      }
    }
  }
  // no CTA goes on (and may leave) while a peer still reads its shared memory
  cluster_sync_all();

  // 4b. between the two clusters of a replica: each leaves its sums in global memory; whichever CTA of a pair
  // (same columns, the two row halves) arrives second adds the two (half 0 + half 1: one addition, the same bits
  // whoever does it) and finishes the update.
  float* mine = scratch + ((int64_t)g * 2 + half) * scratch_stride;
  const float* other = scratch + ((int64_t)g * 2 + (half ^ 1)) * scratch_stride;
#pragma unroll
  for (int i = 0; i < kStepOwn4; ++i) {
    const int e = tid + i * kStepThreads;
    if (e < CT * KO4) __stcg(reinterpret_cast<float4*>(mine + (e / KO4) * K + r * KO + (e % KO4) * 4), sw[i]);
  }
  if (tid < KO4) __stcg(reinterpret_cast<float4*>(mine + CT * K + r * KO + tid * 4), sc);
  if (r == 0 && tid <= CT) __stcg(mine + (CT + 1) * K + tid, ss);
  __threadfence();
  __syncthreads();
  if (tid == 0) is_last = atomicInc(&counters[g * kStepCluster + r], 1u) == 1u ? 1u : 0u;   // wraps back to 0
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  auto finish = [&](float s, float vold, float wold, float& vnew) {      // v <- mu v + G; returns W - eta v
    float step = s;
    if (mu != 0.f) step = fmaf(mu, vold, s);
    vnew = step;
    return fmaf(-lr, step, wold);
  };
#pragma unroll
  for (int i = 0; i < kStepOwn4; ++i) {
    const int e = tid + i * kStepThreads;
    if (e < CT * KO4) {
      const int64_t at = (int64_t)(e / KO4) * K + r * KO + (e % KO4) * 4;
      const float4 s = add4(sw[i], __ldcg(reinterpret_cast<const float4*>(other + at)));
      float4 vn, wn;
      wn.x = finish(s.x, vu[i].x, wu[i].x, vn.x); wn.y = finish(s.y, vu[i].y, wu[i].y, vn.y);
      wn.z = finish(s.z, vu[i].z, wu[i].z, vn.z); wn.w = finish(s.w, vu[i].w, wu[i].w, vn.w);
      if (mu != 0.f) *reinterpret_cast<float4*>(Vg + at) = vn;
      *reinterpret_cast<float4*>(Wg + at) = wn;
      if (Wb != nullptr) {
        __nv_bfloat162 lo = __floats2bfloat162_rn(wn.x, wn.y), hi = __floats2bfloat162_rn(wn.z, wn.w);
        *reinterpret_cast<uint2*>(Wb + (int64_t)g * w_gstride + at) =
            make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
      }
    }
  }
  if (prev_bias) {
    const int k = r * KO + tid * 4;
    const float4 s = add4(sc, __ldcg(reinterpret_cast<const float4*>(other + CT * K + k)));
    const int64_t at = (int64_t)g * w_gstride + k;
    float4 vn, bn;
    bn.x = finish(s.x, vb_prev.x, b_prev.x, vn.x); bn.y = finish(s.y, vb_prev.y, b_prev.y, vn.y);
    bn.z = finish(s.z, vb_prev.z, b_prev.z, vn.z); bn.w = finish(s.w, vb_prev.w, b_prev.w, vn.w);
    if (mu != 0.f) *reinterpret_cast<float4*>(pvbias + at) = vn;
    *reinterpret_cast<float4*>(pbias + at) = bn;
  }
  if (r == 0 && tid <= CT) {
    const float s = ss + __ldcg(other + (CT + 1) * K + tid);
    if (tid == 0) {
      if (loss_out != nullptr) loss_out[g] = s * invB;
    } else if (bias != nullptr) {
      const int64_t at = (int64_t)g * w_gstride + tid - 1;
      float vn;
      const float bn = finish(s, vb_own, b_own, vn);
      if (mu != 0.f) vbias[at] = vn;
      bias[at] = bn;
    }
  }
}

}  // namespace

// floats per (replica, half) of the scratch: G sums [C][K], column sums [K], loss / bias sums
static int64_t step_scratch_stride(int C, int K) { return (int64_t)(C + 1) * K + 32; }

size_t head_step_scratch_bytes(int m, int C, int K) { return (size_t)m * 2 * step_scratch_stride(C, K) * 4; }
size_t head_step_counter_bytes(int m) { return (size_t)m * kStepCluster * 4; }

bool head_step_ok(const HeadStepArgs& a) {
  if (a.C != 10 || a.loss_kind != LS_LOSS_SOFTMAX_CE || a.dPrev == nullptr || a.A == nullptr || a.scratch == nullptr ||
      a.counters == nullptr)
    return false;
  if (a.B % (kStepBlocks * 4) != 0 || a.B / kStepBlocks > kStepMaxRows) return false;
  if (a.K < 128 || a.K % 128 != 0 || a.C * (a.K / kStepCluster) > kStepOwn4 * 4 * kStepThreads)
    return false;
  if (reinterpret_cast<uintptr_t>(a.A) % 16 != 0 || reinterpret_cast<uintptr_t>(a.W) % 16 != 0 || a.w_gstride % 4 != 0 ||
      reinterpret_cast<uintptr_t>(a.dPrev) % 8 != 0)
    return false;
  return step_layout(a.C, a.K, a.B / kStepBlocks).total <= 226 * 1024;
}

int launch_head_step(const HeadStepArgs& a, cudaStream_t st, int64_t* launches) {
  if (!head_step_ok(a)) return cudaErrorInvalidValue;
  auto kern = head_step_kernel<10>;
  static uint64_t configured = 0;        // one bit per device
  {
    cudaError_t e = allow_dynamic_smem(kern, 226 * 1024, &configured);
    if (e != cudaSuccess) return e;
  }
  if (launches) ++*launches;
  const size_t smem = step_layout(a.C, a.K, a.B / kStepBlocks).total;
  return launch_dep(kern, dim3(kStepCluster, kStepBlocks / kStepCluster, (unsigned)a.groups), dim3(kStepThreads), smem, st,
                    kStepCluster, static_cast<const __nv_bfloat16*>(a.A), static_cast<const int32_t*>(a.y), a.y_row_off, a.W,
                    a.V, a.Wb, a.bias, a.vbias, a.w_gstride, static_cast<__nv_bfloat16*>(a.dPrev),
                    a.dPrev ? a.pbias : nullptr, a.pvbias, a.loss_out, a.scratch, step_scratch_stride(a.C, a.K), a.counters,
                    a.B, a.K, a.lr, a.mu);
}

}  // namespace ls
