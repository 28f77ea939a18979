// A whole run of local steps of a small linear model in ONE launch (Section 2, PASGD update rule, the case
// k mod tau != 0 applied tau times): softmax regression or least squares.
//
// Such a model's local step is two launches of a few microseconds each, so a period of tau steps is bound by
// launch latency, not by work.  Here a thread-block cluster of S CTAs owns one replica for the whole call and
// splits the INPUT FEATURES: CTA r keeps columns [k_r, k_r + kw) of W (and of its momentum) in shared memory
// and, every step, brings in the same columns of the replica's mini-batch with asynchronous copies.
//
//   forward   partial logits of the CTA's columns, thread = (sample, 1/8 of the columns), three shuffles;
//             every CTA stores its [B][C] partials into the shared memory of ALL CTAs of the cluster
//             (distributed shared memory), one cluster barrier, then every CTA adds the S partials in rank
//             order (so all CTAs hold the same bits), adds the bias and forms loss and dZ for all samples
//   backward  needs no exchange: G[c][k] = sum_b dZ[b][c] X[b][k] over the batch in index order for the CTA's
//             own columns, thread = (four columns, output c); then v <- mu v + G, W <- W - lr v in shared memory
//   bias      replicated in every CTA, updated identically; rank 0 writes it back
// The only global traffic besides the mini-batches is one read and one write of the replica's state per CALL.
// Clusters are independent of one another (replicas do not interact between averaging steps); inside a cluster
// the only wait is the hardware cluster barrier, once per step (the partials are double-buffered).
// Sums run in a fixed order: results do not depend on scheduling.
#include "ls_internal.h"
#include "tc_ptx.cuh"

namespace ls {
namespace {

using namespace ptx;

constexpr int kThreads = 256;
constexpr int kMaxCluster = 8;
constexpr size_t kSmemCap = 200 * 1024;      // a CTA's share of W (+ v), of one mini-batch, and small vectors

struct PeriodArgs {
  const float* X; const void* y;          // dataset rows [n][K] fp32, labels (int32) or targets (float)
  const int64_t* row_off;                 // device [tau][m]
  float* W; float* V;                     // replica 0's weights [C][K] / momentum; replica stride gstride
  float* bias; float* vbias;              // [C] or null
  int64_t gstride;
  float* loss_out;                        // [tau][m] or null
  int tau, m, B, K, C, kind, S, kw4;      // S CTAs per replica, kw4 = float4 columns per CTA (the last may have fewer)
  int two_x;                              // two mini-batch buffers: the next step's rows are copied during this step
  float lr, mu;
};

__device__ __forceinline__ void cp_async16(void* dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src)
               : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() {
  asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;" ::: "memory");
}

template <int C>
__global__ void __launch_bounds__(kThreads, 1) linear_period_kernel(const PeriodArgs a) {
  extern __shared__ __align__(16) float smem[];
  const int K = a.K, B = a.B, S = a.S, tid = threadIdx.x;
  const int g = blockIdx.x / S, rank = S > 1 ? (int)cluster_ctarank() : 0;
  const bool has_v = a.mu != 0.f;
  const int k40 = rank * a.kw4;                                        // first float4 column of this CTA
  const int n4 = max(0, min(a.kw4, K / 4 - k40));                      // how many it has
  const int kw = a.kw4 * 4;                                            // row pitch of the slices in shared memory
  float* Ws = smem;                              // [C][kw]
  float* Vs = Ws + (size_t)C * kw;               // [C][kw] (momentum; unused without it)
  float* Xs = Vs + (has_v ? (size_t)C * kw : 0); // [B][kw]
  float* recv = Xs + (size_t)B * kw;             // [2][S][B][C] partial logits of every CTA of the cluster (two steps)
  float* dZs = recv + 2 * (size_t)S * B * C;     // [B][C]
  float* rl = dZs + (size_t)B * C;               // [B] per-sample losses
  float* bs = rl + B;                            // [C] bias, [C] its momentum
  long long* offs = reinterpret_cast<long long*>((reinterpret_cast<uintptr_t>(bs + 2 * C) + 7) & ~(uintptr_t)7);   // [tau] first rows of this replica's batches
  float* Xs2 = a.two_x ? reinterpret_cast<float*>((reinterpret_cast<uintptr_t>(offs + a.tau) + 15) & ~(uintptr_t)15)
                       : Xs;                                                     // second mini-batch buffer when it fits
  grid_dep_wait();
  grid_dep_launch();
  for (int s = tid; s < a.tau; s += kThreads) offs[s] = a.row_off[(int64_t)s * a.m + g];
  float* Wg = a.W + (int64_t)g * a.gstride + k40 * 4;
  float* Vg = a.V + (int64_t)g * a.gstride + k40 * 4;
  for (int i = tid; i < C * n4; i += kThreads) {
    const int c = i / n4, j = i - c * n4;
    *reinterpret_cast<float4*>(Ws + (size_t)c * kw + j * 4) = *reinterpret_cast<const float4*>(Wg + (size_t)c * K + j * 4);
    if (has_v)
      *reinterpret_cast<float4*>(Vs + (size_t)c * kw + j * 4) = *reinterpret_cast<const float4*>(Vg + (size_t)c * K + j * 4);
  }
  if (tid < C) {
    bs[tid] = a.bias ? a.bias[(int64_t)g * a.gstride + tid] : 0.f;
    bs[C + tid] = (a.bias && has_v) ? a.vbias[(int64_t)g * a.gstride + tid] : 0.f;
  }
  const int slice = tid & 7, sb = tid >> 3;      // forward: 32 samples per pass, 8 slices of the columns each
  const float invB = 1.0f / (float)B;
  const uint32_t recv_addr = smem_u32(recv);

  auto fetch = [&](int s, float* dst) {          // this CTA's columns of the rows of step s
    const float* Xg = a.X + offs[s] * K + k40 * 4;
    for (int i = tid; i < B * n4; i += kThreads) {
      const int b = i / n4, j = i - b * n4;
      cp_async16(dst + (size_t)b * kw + j * 4, Xg + (size_t)b * K + j * 4);
    }
  };
  __syncthreads();                               // offs, bs, Ws are in place
  if (a.two_x) fetch(0, Xs);
  for (int s = 0; s < a.tau; ++s) {
    const int64_t r0 = offs[s];
    float* Xc = (a.two_x && (s & 1)) ? Xs2 : Xs;
    __syncthreads();                             // the previous step has finished with its buffers
    if (!a.two_x) fetch(s, Xc);
    cp_async_wait_all();
    __syncthreads();
    if (a.two_x && s + 1 < a.tau) fetch(s + 1, (s & 1) ? Xs : Xs2);    // lands while this step computes
    // ---- forward: this CTA's partial logits ---------------------------------------------------------
    // (every CTA WRITES its partials into the shared memory of all its peers: remote stores cost no round trip,
    //  and after the cluster barrier every read is local)
    const uint32_t slot_off = (uint32_t)(((s & 1) * S + rank) * B * C * 4);
    const uint32_t dst_addr = (S > 1 && slice < S ? map_to_rank(recv_addr, (uint32_t)slice) : recv_addr) + slot_off;
    for (int b0 = 0; b0 < B; b0 += kThreads / 8) {
      const int b = b0 + sb;
      float acc[C];
#pragma unroll
      for (int c = 0; c < C; ++c) acc[c] = 0.f;
      if (b < B) {
        const float* xr = Xc + (size_t)b * kw;
        for (int k4 = slice; k4 < n4; k4 += 8) {
          const float4 x = *reinterpret_cast<const float4*>(xr + k4 * 4);
#pragma unroll
          for (int c = 0; c < C; ++c) {
            const float4 w = *reinterpret_cast<const float4*>(Ws + (size_t)c * kw + k4 * 4);
            acc[c] = fmaf(x.x, w.x, fmaf(x.y, w.y, fmaf(x.z, w.z, fmaf(x.w, w.w, acc[c]))));
          }
        }
      }
#pragma unroll
      for (int c = 0; c < C; ++c) {
        acc[c] += __shfl_xor_sync(0xffffffffu, acc[c], 1);
        acc[c] += __shfl_xor_sync(0xffffffffu, acc[c], 2);
        acc[c] += __shfl_xor_sync(0xffffffffu, acc[c], 4);
      }
      // after the shuffles all eight lanes of a sample hold its partial logits: lane r sends them to CTA r
      if (b < B && slice < S) {
#pragma unroll
        for (int c = 0; c < C; ++c)
          asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(dst_addr + (uint32_t)((b * C + c) * 4)), "f"(acc[c]) : "memory");
      }
    }
    if (S > 1) cluster_sync_all(); else __syncthreads();
    // ---- logits = partials in rank order + bias; loss and dZ (every CTA, identically) -----------------
    for (int b = tid; b < B; b += kThreads) {
      float z[C];
      const float* in = recv + (size_t)(s & 1) * S * B * C + b * C;
#pragma unroll
      for (int c = 0; c < C; ++c) z[c] = in[c];
      for (int r = 1; r < S; ++r)
#pragma unroll
        for (int c = 0; c < C; ++c) z[c] += in[(size_t)r * B * C + c];
      if (a.kind == LS_LOSS_SOFTMAX_CE) {
        const int yb = static_cast<const int*>(a.y)[r0 + b];
        float zmax = -INFINITY;
#pragma unroll
        for (int c = 0; c < C; ++c) { z[c] += bs[c]; zmax = fmaxf(zmax, z[c]); }
        float sum = 0.f, zy = 0.f;
#pragma unroll
        for (int c = 0; c < C; ++c) {
          if (c == yb) zy = z[c];
          z[c] = expf(z[c] - zmax);
          sum += z[c];
        }
        rl[b] = zmax + logf(sum) - zy;
        const float inv = 1.0f / sum;
#pragma unroll
        for (int c = 0; c < C; ++c) dZs[b * C + c] = (z[c] * inv - (c == yb ? 1.f : 0.f)) * invB;
      } else {
        const float r = z[0] + bs[0] - static_cast<const float*>(a.y)[r0 + b];
        rl[b] = 0.5f * r * r;
        dZs[b * C] = r * invB;
      }
    }
    __syncthreads();
    if (tid >= kThreads - 32 && rank == 0 && a.loss_out != nullptr) {
      // the last warp (it has the least gradient work): lane l sums rows l, l + 32, ..., then a fixed shuffle tree
      const int l = tid & 31;
      float t = 0.f;
      for (int b = l; b < B; b += 32) t += rl[b];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
      if (l == 0) a.loss_out[(int64_t)s * a.m + g] = t * invB;
    }
    // ---- weight gradient + update of this CTA's columns, in shared memory ----------------------------
    for (int i = tid; i < n4 * C; i += kThreads) {
      const int k4 = i / C, c = i - k4 * C;
      float4 gr = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int b = 0; b < B; ++b) {
        const float4 x = *reinterpret_cast<const float4*>(Xc + (size_t)b * kw + k4 * 4);
        const float d = dZs[b * C + c];
        gr.x = fmaf(d, x.x, gr.x); gr.y = fmaf(d, x.y, gr.y); gr.z = fmaf(d, x.z, gr.z); gr.w = fmaf(d, x.w, gr.w);
      }
      float4* wp = reinterpret_cast<float4*>(Ws + (size_t)c * kw + k4 * 4);
      float4 w = *wp, st = gr;
      if (has_v) {
        float4* vp = reinterpret_cast<float4*>(Vs + (size_t)c * kw + k4 * 4);
        const float4 v = *vp;
        st = make_float4(fmaf(a.mu, v.x, st.x), fmaf(a.mu, v.y, st.y), fmaf(a.mu, v.z, st.z), fmaf(a.mu, v.w, st.w));
        *vp = st;
      }
      w.x = fmaf(-a.lr, st.x, w.x); w.y = fmaf(-a.lr, st.y, w.y); w.z = fmaf(-a.lr, st.z, w.z); w.w = fmaf(-a.lr, st.w, w.w);
      *wp = w;
    }
    // the bias is read again only after the barrier at the top of the loop
    if (tid >= kThreads - 64 && tid < kThreads - 64 + C && a.bias != nullptr) {
      const int c = tid - (kThreads - 64);
      float g0 = 0.f, g1 = 0.f, g2 = 0.f, g3 = 0.f;          // four chains, joined in a fixed order
      int b = 0;
      for (; b + 4 <= B; b += 4) {
        g0 += dZs[b * C + c]; g1 += dZs[(b + 1) * C + c]; g2 += dZs[(b + 2) * C + c]; g3 += dZs[(b + 3) * C + c];
      }
      for (; b < B; ++b) g0 += dZs[b * C + c];
      const float gb = (g0 + g1) + (g2 + g3);
      float st = gb;
      if (has_v) { st = fmaf(a.mu, bs[C + c], gb); bs[C + c] = st; }
      bs[c] = fmaf(-a.lr, st, bs[c]);
    }
  }
  __syncthreads();
  for (int i = tid; i < C * n4; i += kThreads) {
    const int c = i / n4, j = i - c * n4;
    *reinterpret_cast<float4*>(Wg + (size_t)c * K + j * 4) = *reinterpret_cast<const float4*>(Ws + (size_t)c * kw + j * 4);
    if (has_v)
      *reinterpret_cast<float4*>(Vg + (size_t)c * K + j * 4) = *reinterpret_cast<const float4*>(Vs + (size_t)c * kw + j * 4);
  }
  if (tid < C && rank == 0 && a.bias != nullptr) {
    a.bias[(int64_t)g * a.gstride + tid] = bs[tid];
    if (has_v) a.vbias[(int64_t)g * a.gstride + tid] = bs[C + tid];
  }
  // no CTA leaves while a peer may still write partials into its shared memory
  if (S > 1) cluster_sync_all();
}

// CTAs per replica: as many as leave every CTA at least 16 float4 columns, up to the portable cluster size
int cluster_for(int K) {
  int s = (K / 4) / 16;
  return s < 1 ? 1 : (s > kMaxCluster ? kMaxCluster : s);
}
size_t smem_bytes(int B, int K, int C, bool has_v, int tau, bool two_x) {
  const int S = cluster_for(K), kw = ((K / 4 + S - 1) / S) * 4;
  return ((size_t)C * kw * (has_v ? 2 : 1) + (size_t)B * kw * (two_x ? 2 : 1) + (2 * S + 1) * (size_t)B * C + B + 2 * C + 2) *
             sizeof(float) + (size_t)tau * 8 + 32;
}

template <int C>
int launch_c(const PeriodArgs& a, size_t smem, cudaStream_t st) {
  static uint64_t configured = 0;
  cudaError_t e = allow_dynamic_smem(linear_period_kernel<C>, (int)kSmemCap, &configured);
  if (e != cudaSuccess) return e;
  return launch_dep(linear_period_kernel<C>, dim3((unsigned)(a.m * a.S)), dim3(kThreads), smem, st, (unsigned)a.S, a);
}

}  // namespace

// A one-layer fp32 model with 10 or 1 outputs (the instantiated counts) and a feature count that is a multiple of
// 4 (16-byte copies), whose per-CTA share of the weights and of one mini-batch fits in shared memory.
bool linear_period_ok(int B, int K, int C, bool has_v) {
  return (C == 10 || C == 1) && K >= 4 && K % 4 == 0 && B >= 1 && B <= LS_MAX_BATCH &&
         smem_bytes(B, K, C, has_v, kRowOffCap, false) <= kSmemCap;
}

int launch_linear_period(const float* X, const void* y, const int64_t* row_off, float* W, float* V, float* bias,
                         float* vbias, int64_t gstride, float* loss_out, int tau, int m, int B, int K, int C, int kind,
                         float lr, float mu, cudaStream_t st, int64_t* launches) {
  if (!linear_period_ok(B, K, C, mu != 0.f) || reinterpret_cast<uintptr_t>(X) % 16 != 0 || gstride % 4 != 0)
    return cudaErrorInvalidValue;
  if (tau < 1 || tau > kRowOffCap) return cudaErrorInvalidValue;
  const int S = cluster_for(K);
  const bool two_x = smem_bytes(B, K, C, mu != 0.f, tau, true) <= kSmemCap;
  PeriodArgs a{X, y, row_off, W, V, bias, vbias, gstride, loss_out, tau, m, B, K, C, kind, S, (K / 4 + S - 1) / S,
               two_x ? 1 : 0, lr, mu};
  const size_t smem = smem_bytes(B, K, C, mu != 0.f, tau, two_x);
  if (launches) ++*launches;
  return C == 10 ? launch_c<10>(a, smem, st) : launch_c<1>(a, smem, st);
}

}  // namespace ls
