// Per-node SGD chains on CSR rows (Eq. 5 on the paper's kind of data: a few tens of features per
// row in a very wide model). One warp per node, one lane per nonzero.
//
// The model of node j is held as w = s * u with an fp64 scalar s: the regulariser's factor
// (1 - eta_n lambda) multiplies s only, and the loss term touches the row's nonzeros only:
//     z = s (u . x);  g = L'(y, z);  s' = s (1 - eta_n lambda);  u_c <- u_c - (eta_n g / s') x_c.
// These are the iterates of Eq. 5 exactly (in exact arithmetic). s stays fp64 because eta_n lambda
// can be far below the fp32 rounding step of 1.
//
// Latency hiding: the sample stream is known in advance, so the row extents (two row_ptr entries and
// the label) of step s+2P and the column/value segments of step s+P are already in registers when
// step s starts; only the gather of u, the warp reduction and the scatter are on the serial path.
#pragma once

#include "common.cuh"

namespace wpsgd {

struct CsrParams {
  const long long* row_ptr;
  const int* col_idx;
  const float* val;
  const float* y;
  const long long* shard_off;
  const long long* n_steps;
  const long long* first;  // steps every node has already run (continued chains), or null
  const long long* idx_off;
  const uint32_t* idx;
  const int* order;
  float* U;        // [k, d] unscaled models
  double* scale;   // [k]
  int k;
  long long d;
  float eta0;
  int sched;
  float lambda;
  int loss;
  int resume;  // 1: continue from the models and scales the context holds
  DevStatus* status;
};

// u rows <- w0 (or zeros) unless keep_models, scale <- 1
__global__ void csr_init_kernel(float* __restrict__ U, double* __restrict__ scale, const float* __restrict__ w0, int k,
                                long long d, int keep_models) {
  const long long total = (long long)k * d;
  if (!keep_models)
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x)
      U[i] = w0 ? w0[i % d] : 0.0f;
  if (blockIdx.x == 0)
    for (int j = threadIdx.x; j < k; j += blockDim.x) scale[j] = 1.0;
}

template <int P>
__global__ void __launch_bounds__(32) chain_csr_kernel(const CsrParams p) {
  constexpr int Q = 2;  // nonzeros per lane kept in registers (rows up to 64 nonzeros); longer rows loop
  const int lane = threadIdx.x;
  const int j = p.order[blockIdx.x];
  const long long n_run = p.n_steps[j];
  const long long* rp = p.row_ptr + p.shard_off[j];
  const float* yshard = p.y + p.shard_off[j];
  const uint32_t* idx = p.idx + p.idx_off[j];
  float* u = p.U + (size_t)j * p.d;
  // The scale factor does not depend on the data: s_n = prod_{q<=n} (1 - eta_q lambda). It is advanced in fp64
  // ahead of the chain, together with the rows, and handed to the step as two floats (s before the step, and
  // eta_n / s after it), so that no fp64 division or square root sits on the serial path.
  double sc = p.resume ? p.scale[j] : 1.0;  // scale after the last step whose constants have been prepared
  const long long first = p.resume ? p.first[j] : 0;
  const double lam = (double)p.lambda, eta0 = (double)p.eta0;
  auto prepare_scalars = [&](long long step0, float& s_before, float& eta_over_s, float& fold) {
    fold = 0.0f;
    if (sc < 1e-12) {  // fold the scale into u at this step, before fp32 range is at risk
      fold = (float)sc;
      sc = 1.0;
    }
    s_before = (float)sc;
    const double eta = p.sched == LR_INV_SQRT ? eta0 / sqrt((double)(first + step0 + 1)) : eta0;
    sc *= (1.0 - eta * lam);
    eta_over_s = (float)(eta / sc);
  };

  // rings (slot = step mod P): sample id of step s+3P; extents+label of step s+2P... see refill below
  uint32_t ib[P];
  long long ra0[P], ra1[P];
  float ya[P];
  long long sb[P];
  int nb[P];
  float yb[P];
  int cb[P][Q];
  float vb[P][Q];
  float scb[P], cfb[P], fob[P];

  // prologue: bring the three pipeline levels up (dependent loads, paid once)
#pragma unroll
  for (int t = 0; t < P; ++t) {
    ib[t] = 0u; ra0[t] = 0; ra1[t] = 0; ya[t] = 0.0f; sb[t] = 0; nb[t] = 0; yb[t] = 0.0f;
    scb[t] = 1.0f; cfb[t] = 0.0f; fob[t] = 0.0f;
#pragma unroll
    for (int q = 0; q < Q; ++q) { cb[t][q] = 0; vb[t][q] = 0.0f; }
    if (t < n_run) {
      const uint32_t i0 = idx[t];
      const long long b = rp[i0], e = rp[i0 + 1];
      sb[t] = b; nb[t] = (int)(e - b); yb[t] = yshard[i0];
      prepare_scalars(t, scb[t], cfb[t], fob[t]);
#pragma unroll
      for (int q = 0; q < Q; ++q) {
        const int o = lane + 32 * q;
        if (o < nb[t]) { cb[t][q] = p.col_idx[b + o]; vb[t][q] = p.val[b + o]; }
      }
    }
    if (t + P < n_run) {
      const uint32_t i1 = idx[t + P];
      ra0[t] = rp[i1]; ra1[t] = rp[i1 + 1]; ya[t] = yshard[i1];
    }
    if (t + 2 * P < n_run) ib[t] = idx[t + 2 * P];
  }

  for (long long s0 = 0; s0 < n_run; s0 += P) {
#pragma unroll
    for (int t = 0; t < P; ++t) {
      const long long s = s0 + t;
      if (s >= n_run) break;
      // ---- this step's row, out of the ring ------------------------------------------------------
      const long long beg = sb[t];
      const int nnz = nb[t];
      const float yv = yb[t];
      int c[Q];
      float v[Q];
#pragma unroll
      for (int q = 0; q < Q; ++q) { c[q] = cb[t][q]; v[q] = vb[t][q]; }
      const float s_before = scb[t], eta_over_s = cfb[t], fold = fob[t];
      if (fold != 0.0f) {  // rare: the scale was folded back at this step
        for (long long cc = lane; cc < p.d; cc += 32) u[cc] *= fold;
        __syncwarp();
      }
      // ---- margin -------------------------------------------------------------------------------
      float uq[Q];
#pragma unroll
      for (int q = 0; q < Q; ++q) uq[q] = (lane + 32 * q < nnz) ? u[c[q]] : 0.0f;  // gathers in flight ...
      // ---- ... while the three levels of slot t are refilled ------------------------------------------------------
      if (s + P < n_run) {
        const long long b = ra0[t];
        const int cnt = (int)(ra1[t] - b);
        sb[t] = b; nb[t] = cnt; yb[t] = ya[t];
        prepare_scalars(s + P, scb[t], cfb[t], fob[t]);
#pragma unroll
        for (int q = 0; q < Q; ++q) {
          const int o = lane + 32 * q;
          if (o < cnt) { cb[t][q] = p.col_idx[b + o]; vb[t][q] = p.val[b + o]; }
        }
      }
      if (s + 2 * P < n_run) {
        const uint32_t i2 = ib[t];
        ra0[t] = rp[i2]; ra1[t] = rp[i2 + 1]; ya[t] = yshard[i2];
      }
      if (s + 3 * P < n_run) ib[t] = idx[s + 3 * P];

      float acc = 0.0f;
#pragma unroll
      for (int q = 0; q < Q; ++q) acc = fmaf(uq[q], v[q], acc);
      for (int o = lane + 32 * Q; o < nnz; o += 32) acc = fmaf(u[p.col_idx[beg + o]], p.val[beg + o], acc);
      acc = warp_sum(acc);
      const float z = s_before * acc;
      const float g = loss_derivative(p.loss, yv, z);
      // ---- loss term on the row's nonzeros: u_c <- u_c - (eta_n g / s_n) x_c -----------------------------
      if (g != 0.0f) {
        const float coef = eta_over_s * g;
#pragma unroll
        for (int q = 0; q < Q; ++q)
          if (lane + 32 * q < nnz) u[c[q]] = fmaf(-coef, v[q], uq[q]);
        for (int o = lane + 32 * Q; o < nnz; o += 32) {
          const int cc = p.col_idx[beg + o];
          u[cc] = fmaf(-coef, p.val[beg + o], u[cc]);
        }
      }
      __syncwarp();  // the next step's gathers must see this step's scatters
    }
  }
  if (lane == 0) p.scale[j] = sc;
}

}  // namespace wpsgd
