// Per-node SGD chains on dense rows (Algorithm 1, inner loop; Eq. 5), direct form: one step per
// sample, z = w.x, g = L'(y, z), w <- w - eta (lambda w + g x).
//
// Two kernels:
//   chain_reg_kernel      the model lives in registers, split over a CTA (one node per CTA) or
//                         over one warp (one node per warp, several nodes per CTA). Rows of the
//                         next PF steps are already in flight (register ring) when a step starts:
//                         their addresses are known in advance because the sample stream does not
//                         depend on w.
//   chain_generic_kernel  any d, any row stride, any alignment: scalar strided loops, the model
//                         kept in its row of W (each element is only ever touched by one thread).
#pragma once

#include "common.cuh"

namespace wpsgd {

struct ChainParams {
  const void* X;               // [N, ld] row-major
  long long ld;                // row stride in elements
  const float* y;              // [N]
  const long long* shard_off;  // [k+1]
  const long long* n_steps;    // [k] steps to run in this launch
  const long long* first;      // [k] steps already run (step numbers continue from here)
  const long long* idx_off;    // [k+1] offsets into idx
  const uint32_t* idx;         // sample stream of this launch
  const int* order;            // [k] node ids, longest chain first
  float* W;                    // [k, d] models
  const float* w0;             // [d] or nullptr
  int resume;                  // 1: start from W (continue), 0: start from w0 / zeros
  int k;
  long long d;
  float eta0;
  int sched;
  float lambda;
  int loss;
  DevStatus* status;
};

template <typename XT, int R, int PF, bool BLOCK_PER_NODE>
__global__ void __launch_bounds__(BLOCK_PER_NODE ? 512 : 128)
chain_reg_kernel(const ChainParams p) {
  constexpr int V = XVec<XT>::V;
  __shared__ float red[2][32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int nwarps = blockDim.x >> 5;
  const int slot = BLOCK_PER_NODE ? (int)blockIdx.x : (int)blockIdx.x * nwarps + warp;
  if (slot >= p.k) return;
  const int j = p.order[slot];
  const int tid = BLOCK_PER_NODE ? (int)threadIdx.x : lane;
  const int T = BLOCK_PER_NODE ? (int)blockDim.x : 32;
  const long long n_run = p.n_steps[j];
  const long long n_first = p.first[j];
  const long long d = p.d;
  const char* shard = (const char*)p.X + (size_t)p.shard_off[j] * (size_t)p.ld * sizeof(XT);
  const float* yshard = p.y + p.shard_off[j];
  const uint32_t* idx = p.idx + p.idx_off[j];
  const size_t row_bytes = (size_t)p.ld * sizeof(XT);

  // ---- initial model -------------------------------------------------------------------------------
  float w[R][V];
  bool act[R];
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const long long c0 = ((long long)r * T + tid) * V;
    act[r] = c0 < d;
#pragma unroll
    for (int v = 0; v < V; ++v) w[r][v] = 0.0f;
    if (act[r]) {
      const float* src = p.resume ? (p.W + (size_t)j * d + c0) : (p.w0 ? p.w0 + c0 : nullptr);
      if (src) {
#pragma unroll
        for (int v = 0; v < V; ++v) w[r][v] = src[v];
      }
    }
  }

  // ---- register ring: rows of steps s .. s+PF-1, sample ids of steps s+PF .. s+2PF-1 -----------------
  uint4 xb[PF][R];
  float yb[PF];
  uint32_t ib[PF];
#pragma unroll
  for (int u = 0; u < PF; ++u) {
    yb[u] = 0.0f;
    ib[u] = 0u;
#pragma unroll
    for (int r = 0; r < R; ++r) xb[u][r] = make_uint4(0u, 0u, 0u, 0u);
    if (u < n_run) {
      const uint32_t i0 = idx[u];
      const char* row = shard + (size_t)i0 * row_bytes;
#pragma unroll
      for (int r = 0; r < R; ++r)
        if (act[r]) xb[u][r] = ld_stream16(row + ((size_t)r * T + tid) * 16);
      yb[u] = yshard[i0];
    }
    if (u + PF < n_run) ib[u] = idx[u + PF];
  }

  const float lam = p.lambda;
  for (long long s0 = 0; s0 < n_run; s0 += PF) {
#pragma unroll
    for (int u = 0; u < PF; ++u) {
      const long long s = s0 + u;
      if (s >= n_run) break;
      // take this step's row out of the ring and refill the slot with the row of step s+PF
      float x[R][V];
#pragma unroll
      for (int r = 0; r < R; ++r) XVec<XT>::widen(xb[u][r], x[r]);
      const float yv = yb[u];
      if (s + PF < n_run) {
        const uint32_t i1 = ib[u];
        const char* row = shard + (size_t)i1 * row_bytes;
#pragma unroll
        for (int r = 0; r < R; ++r)
          if (act[r]) xb[u][r] = ld_stream16(row + ((size_t)r * T + tid) * 16);
        yb[u] = yshard[i1];
      }
      if (s + 2 * PF < n_run) ib[u] = idx[s + 2 * PF];

      // margin z = w . x
      float acc[R];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        acc[r] = 0.0f;
#pragma unroll
        for (int v = 0; v < V; ++v) acc[r] = fmaf(w[r][v], x[r][v], acc[r]);
      }
#pragma unroll
      for (int r = 1; r < R; ++r) acc[0] += acc[r];
      float z = warp_sum(acc[0]);
      if (BLOCK_PER_NODE && nwarps > 1) {
        const int par = (int)(s & 1);
        if (lane == 0) red[par][warp] = z;
        __syncthreads();
        z = 0.0f;
        for (int i = 0; i < nwarps; ++i) z += red[par][i];
      }
      const float eta = step_size(p.eta0, p.sched, n_first + s + 1);
      const float g = loss_derivative(p.loss, yv, z);
      const float neg_el = -eta * lam, neg_eg = -eta * g;
      // w <- (w - eta lambda w) - eta g x, with the small factor applied by FMA so that
      // 1 - eta lambda is never rounded to fp32
#pragma unroll
      for (int r = 0; r < R; ++r)
#pragma unroll
        for (int v = 0; v < V; ++v) w[r][v] = fmaf(neg_eg, x[r][v], fmaf(neg_el, w[r][v], w[r][v]));
    }
  }

#pragma unroll
  for (int r = 0; r < R; ++r) {
    const long long c0 = ((long long)r * T + tid) * V;
    if (act[r]) {
      float* dst = p.W + (size_t)j * d + c0;
#pragma unroll
      for (int v = 0; v < V; ++v) dst[v] = w[r][v];
    }
  }
}

// Any shape. One CTA per node, w kept in W[j] (element c is only touched by thread c mod blockDim).
template <typename XT>
__global__ void __launch_bounds__(256) chain_generic_kernel(const ChainParams p) {
  __shared__ float red[2][32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  const int j = p.order[blockIdx.x];
  const long long n_run = p.n_steps[j], n_first = p.first[j], d = p.d;
  const XT* shard = (const XT*)p.X + (size_t)p.shard_off[j] * (size_t)p.ld;
  const float* yshard = p.y + p.shard_off[j];
  const uint32_t* idx = p.idx + p.idx_off[j];
  float* w = p.W + (size_t)j * d;
  if (!p.resume)
    for (long long c = threadIdx.x; c < d; c += blockDim.x) w[c] = p.w0 ? p.w0[c] : 0.0f;
  for (long long s = 0; s < n_run; ++s) {
    const uint32_t i0 = idx[s];
    const XT* row = shard + (size_t)i0 * (size_t)p.ld;
    float acc = 0.0f;
    for (long long c = threadIdx.x; c < d; c += blockDim.x) acc = fmaf(w[c], widen_scalar<XT>(row[c]), acc);
    float z = warp_sum(acc);
    const int par = (int)(s & 1);
    if (lane == 0) red[par][warp] = z;
    __syncthreads();
    z = 0.0f;
    for (int i = 0; i < nwarps; ++i) z += red[par][i];
    const float eta = step_size(p.eta0, p.sched, n_first + s + 1);
    const float g = loss_derivative(p.loss, yshard[i0], z);
    const float neg_el = -eta * p.lambda, neg_eg = -eta * g;
    for (long long c = threadIdx.x; c < d; c += blockDim.x)
      w[c] = fmaf(neg_eg, widen_scalar<XT>(row[c]), fmaf(neg_el, w[c], w[c]));
  }
}

}  // namespace wpsgd
