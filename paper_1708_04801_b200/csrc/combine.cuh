// Aggregation step of Algorithm 1 (v = sum_j weight_j w_j with the weights of Eq. 6 / Eq. 8), model
// export, model broadcast, and the evaluation measures of the paper's experiments.
#pragma once

#include "common.cuh"

namespace wpsgd {

// v[c] = sum_j (weight_j * scale_j) * W[j][c], j ascending, fp64 accumulation. scale may be null.
__global__ void combine_kernel(const float* __restrict__ W, const double* __restrict__ weights,
                               const double* __restrict__ scale, int k, long long d, float* __restrict__ v) {
  for (long long c = (long long)blockIdx.x * blockDim.x + threadIdx.x; c < d; c += (long long)gridDim.x * blockDim.x) {
    double a = 0.0;
    int j = 0;
    for (; j + 4 <= k; j += 4) {
      const float f0 = W[(size_t)(j + 0) * d + c], f1 = W[(size_t)(j + 1) * d + c];
      const float f2 = W[(size_t)(j + 2) * d + c], f3 = W[(size_t)(j + 3) * d + c];
      // the k effective weights are the same for every thread: broadcast loads that stay in L1
      a = fma(weights[j + 0] * (scale ? scale[j + 0] : 1.0), (double)f0, a);
      a = fma(weights[j + 1] * (scale ? scale[j + 1] : 1.0), (double)f1, a);
      a = fma(weights[j + 2] * (scale ? scale[j + 2] : 1.0), (double)f2, a);
      a = fma(weights[j + 3] * (scale ? scale[j + 3] : 1.0), (double)f3, a);
    }
    for (; j < k; ++j) a = fma(weights[j] * (scale ? scale[j] : 1.0), (double)W[(size_t)j * d + c], a);
    v[c] = (float)a;
  }
}

// W_out[j][c] = scale_j * W[j][c]
__global__ void export_models_kernel(const float* __restrict__ W, const double* __restrict__ scale, int k, long long d,
                                     float* __restrict__ out) {
  const long long total = (long long)k * d;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x)
    out[i] = scale ? (float)(scale[i / d] * (double)W[i]) : W[i];
}

// W[j][:] = v for every node; scale_j = 1
__global__ void broadcast_model_kernel(float* __restrict__ W, double* __restrict__ scale, const float* __restrict__ v,
                                       int k, long long d) {
  const long long total = (long long)k * d;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x)
    W[i] = v[i % d];
  if (blockIdx.x == 0)
    for (int j = threadIdx.x; j < k; j += blockDim.x) scale[j] = 1.0;
}

// Pass 1 of the objective (Eq. 3-4): one warp per row, per-block partial sums of the loss and of the
// misclassification count, written to part[2 * blockIdx.x + {0,1}] (fixed order -> deterministic).
template <typename XT>
__global__ void __launch_bounds__(256) objective_rows_kernel(const XT* __restrict__ X, long long ld,
                                                             const float* __restrict__ y, long long n_rows,
                                                             const float* __restrict__ w, long long d, int loss,
                                                             double* __restrict__ part) {
  __shared__ double sl[8], se[8];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  double lsum = 0.0, esum = 0.0;
  for (long long i = (long long)blockIdx.x * 8 + warp; i < n_rows; i += (long long)gridDim.x * 8) {
    const XT* row = X + (size_t)i * ld;
    float acc = 0.0f;
    for (long long c = lane; c < d; c += 32) acc = fmaf(w[c], widen_scalar<XT>(row[c]), acc);
    const float z = warp_sum(acc);
    const float yy = y[i];
    double L;
    if (loss == LOSS_HINGE) L = fmax(0.0, 1.0 - (double)yy * (double)z);
    else if (loss == LOSS_LOGISTIC) {
      const double t = (double)yy * (double)z;
      L = t > 0 ? log1p(exp(-t)) : -t + log1p(exp(t));
    } else L = 0.5 * ((double)z - (double)yy) * ((double)z - (double)yy);
    lsum += L;
    esum += ((z >= 0.0f) != (yy >= 0.0f)) ? 1.0 : 0.0;
  }
  if (lane == 0) { sl[warp] = lsum; se[warp] = esum; }
  __syncthreads();
  if (threadIdx.x == 0) {
    double a = 0.0, b = 0.0;
    for (int i = 0; i < 8; ++i) { a += sl[i]; b += se[i]; }
    part[2 * blockIdx.x] = a;
    part[2 * blockIdx.x + 1] = b;
  }
}

// Pass 1 on CSR rows: one warp per row, lanes over the row's nonzeros.
__global__ void __launch_bounds__(256) objective_rows_csr_kernel(const long long* __restrict__ row_ptr,
                                                                 const int* __restrict__ col_idx,
                                                                 const float* __restrict__ val,
                                                                 const float* __restrict__ y, long long n_rows,
                                                                 const float* __restrict__ w, int loss,
                                                                 double* __restrict__ part) {
  __shared__ double sl[8], se[8];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  double lsum = 0.0, esum = 0.0;
  for (long long i = (long long)blockIdx.x * 8 + warp; i < n_rows; i += (long long)gridDim.x * 8) {
    const long long b = row_ptr[i], e = row_ptr[i + 1];
    float acc = 0.0f;
    for (long long q = b + lane; q < e; q += 32) acc = fmaf(w[col_idx[q]], val[q], acc);
    const float z = warp_sum(acc);
    const float yy = y[i];
    double L;
    if (loss == LOSS_HINGE) L = fmax(0.0, 1.0 - (double)yy * (double)z);
    else if (loss == LOSS_LOGISTIC) {
      const double t = (double)yy * (double)z;
      L = t > 0 ? log1p(exp(-t)) : -t + log1p(exp(t));
    } else L = 0.5 * ((double)z - (double)yy) * ((double)z - (double)yy);
    lsum += L;
    esum += ((z >= 0.0f) != (yy >= 0.0f)) ? 1.0 : 0.0;
  }
  if (lane == 0) { sl[warp] = lsum; se[warp] = esum; }
  __syncthreads();
  if (threadIdx.x == 0) {
    double a = 0.0, b2 = 0.0;
    for (int i = 0; i < 8; ++i) { a += sl[i]; b2 += se[i]; }
    part[2 * blockIdx.x] = a;
    part[2 * blockIdx.x + 1] = b2;
  }
}

// Pass 2: out[0] = (lambda/2)|w|^2 + sum(part loss)/n_rows, out[1] = sum(part err)/n_rows. One block.
__global__ void __launch_bounds__(256) objective_finish_kernel(const double* __restrict__ part, int n_part,
                                                               const float* __restrict__ w, long long d, float lambda,
                                                               long long n_rows, double* __restrict__ out) {
  __shared__ double sh[3][256];
  double a = 0.0, b = 0.0, r = 0.0;
  for (int i = threadIdx.x; i < n_part; i += 256) { a += part[2 * i]; b += part[2 * i + 1]; }
  for (long long c = threadIdx.x; c < d; c += 256) r += (double)w[c] * (double)w[c];
  sh[0][threadIdx.x] = a; sh[1][threadIdx.x] = b; sh[2][threadIdx.x] = r;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if (threadIdx.x < o)
      for (int q = 0; q < 3; ++q) sh[q][threadIdx.x] += sh[q][threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const double n = n_rows > 0 ? (double)n_rows : 1.0;
    out[0] = 0.5 * (double)lambda * sh[2][0] + (n_rows > 0 ? sh[0][0] / n : 0.0);
    out[1] = n_rows > 0 ? sh[1][0] / n : 0.0;
  }
}

// Read-only check of a CSR matrix before it is handed to the chains: row_ptr within [0, nnz] and non-decreasing,
// every column in [0, d), columns strictly increasing within a row (so no column occurs twice: the sparse update
// writes every nonzero's model entry once). The first problem found goes to the status word (where = 31 row extents,
// 32 column range, 33 column order; detail = the row). Nothing is read outside [0, nnz).
__global__ void validate_csr_kernel(const long long* __restrict__ row_ptr, const int* __restrict__ col_idx, long long n_rows,
                                    long long nnz, long long d, DevStatus* status) {
  const int lane = threadIdx.x & 31;
  const long long warp0 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long i = warp0; i < n_rows; i += nwarps) {
    const long long b = row_ptr[i], e = row_ptr[i + 1];
    if (b < 0 || e < b || e > nnz) {
      if (lane == 0) set_status(status, DEV_BOUNDS, 31, i);
      continue;
    }
    for (long long q = b + lane; q < e; q += 32) {
      const long long c = col_idx[q];
      if (c < 0 || c >= d) set_status(status, DEV_BOUNDS, 32, i);
      else if (q > b && (long long)col_idx[q - 1] >= c) set_status(status, DEV_BOUNDS, 33, i);
    }
  }
}

}  // namespace wpsgd
