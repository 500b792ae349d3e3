// Per-node SGD chains on dense rows, blocked form (constant step size).
//
// Eq. 5 is a strictly serial recurrence, w_n = a w_{n-1} - eta g_n x_n with a = 1 - eta lambda and
// g_n = L'(y_n, w_{n-1}.x_n). Taking B consecutive samples x_0..x_{B-1} of a chain together and unrolling,
//     w after n samples  = a^n ( w_0 - sum_{m<n} beta_m x_m ),       beta_m = eta g_m / a^{m+1},
//     margin of sample n = a^n ( p_n - sum_{m<n} beta_m G_mn ),      p_n = w_0.x_n,  G_mn = x_m.x_n,
//     w after the block  = w_0 - (1 - a^B) w_0 - sum_m gamma_m x_m,  gamma_m = eta g_m a^{B-1-m}.
// These are the iterates of Eq. 5 exactly (in exact arithmetic; floating point only reassociates).
// p and G are long dot products with no dependency between them, so they run at full issue rate; G does
// not depend on the model at all, so it is computed one block ahead. What stays serial is a scalar
// recurrence of B steps per block, done by one warp.
//
// One CTA per node: warp 0 is the "serial warp" (sums the partial products, runs the B-step
// recurrence, publishes gamma); the other warps are "math warps", each thread owning fixed columns of
// the model (in registers) for the whole chain. Rows reach shared memory through a ring of S blocks
// filled by per-thread 16-byte asynchronous copies: every thread copies exactly the bytes it later
// reads itself, so the ring needs no barrier and no wait that could hang.
//
// Per block b:   math warps                               serial warp
//                p_b partials (needs w)  -> smem          sum G_b partials (written last round)
//                ------------------------- barrier 1 --------------------------------------
//                G_{b+1} partials -> smem                 sum p_b, B-step recurrence, gamma -> smem
//                ------------------------- barrier 2 --------------------------------------
//                w <- w - (1-a^B) w - sum gamma_m x_m     prefetch labels
//                prefetch rows of block b+S
#pragma once

#include "chain_dense.cuh"
#include "common.cuh"

namespace wpsgd {

struct BlockParams {
  ChainParams c;
  int stages;        // S: blocks in the shared-memory ring (>= 2)
  double eta_lambda; // eta * lambda in fp64
};

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
  const uint32_t s = (uint32_t)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(s), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async4(void* smem_dst, const void* gmem_src) {
  const uint32_t s = (uint32_t)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(s), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
// wait until at most `pending` of this thread's committed groups are still in flight (pending in 0..3)
__device__ __forceinline__ void cp_async_wait(int pending) {
  switch (pending) {
    case 0: asm volatile("cp.async.wait_group 0;" ::: "memory"); break;
    case 1: asm volatile("cp.async.wait_group 1;" ::: "memory"); break;
    case 2: asm volatile("cp.async.wait_group 2;" ::: "memory"); break;
    default: asm volatile("cp.async.wait_group 3;" ::: "memory"); break;
  }
}

// dL/dz with the fast exponential and reciprocal units (relative error of a few 2^-22)
template <int LOSS>
__device__ __forceinline__ float loss_derivative_fast(float y, float z) {
  if (LOSS == LOSS_HINGE) return (y * z < 1.0f) ? -y : 0.0f;
  if (LOSS == LOSS_LOGISTIC) return __fdividef(-y, 1.0f + __expf(y * z));
  return z - y;
}

// Quad q (4 consecutive columns) of a 16-byte chunk, widened to fp32.
template <typename XT>
__device__ __forceinline__ void widen_quad(const uint4& raw, int q, float (&f)[4]);
template <>
__device__ __forceinline__ void widen_quad<float>(const uint4& raw, int, float (&f)[4]) {
  f[0] = __uint_as_float(raw.x); f[1] = __uint_as_float(raw.y);
  f[2] = __uint_as_float(raw.z); f[3] = __uint_as_float(raw.w);
}
template <>
__device__ __forceinline__ void widen_quad<__nv_bfloat16>(const uint4& raw, int q, float (&f)[4]) {
  const uint32_t a = q ? raw.z : raw.x, b = q ? raw.w : raw.y;
  f[0] = __uint_as_float(a << 16); f[1] = __uint_as_float(a & 0xffff0000u);
  f[2] = __uint_as_float(b << 16); f[3] = __uint_as_float(b & 0xffff0000u);
}

// Sum of each of 32 per-lane values over the warp; afterwards lane l holds the total of value l.
// 31 shuffles: in every round a lane hands half of its values to its partner and keeps the other half.
__device__ __forceinline__ float warp_transpose_sum32(float (&v)[32]) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int half = 16; half >= 1; half >>= 1) {
    const bool hi = (lane & half) != 0;
#pragma unroll
    for (int i = 0; i < half; ++i) {
      const float send = hi ? v[i] : v[i + half];
      const float keep = hi ? v[i + half] : v[i];
      v[i] = keep + __shfl_xor_sync(0xffffffffu, send, half);
    }
  }
  return v[0];
}

// Same for 8 values: afterwards every lane l holds the total of value l >> 2.
__device__ __forceinline__ float warp_transpose_sum8(float (&v)[8]) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int half = 4; half >= 1; half >>= 1) {
    const int mask = half * 4;  // lane bits 4, 3, 2
    const bool hi = (lane & mask) != 0;
#pragma unroll
    for (int i = 0; i < half; ++i) {
      const float send = hi ? v[i] : v[i + half];
      const float keep = hi ? v[i + half] : v[i];
      v[i] = keep + __shfl_xor_sync(0xffffffffu, send, mask);
    }
  }
  float t = v[0];
  t += __shfl_xor_sync(0xffffffffu, t, 2);
  t += __shfl_xor_sync(0xffffffffu, t, 1);
  return t;
}

constexpr int BLK_B = 8;                           // samples per block
constexpr int BLK_PAIRS = BLK_B * (BLK_B - 1) / 2;  // 28 Gram entries below the diagonal
constexpr int BLK_MAX_MATH_WARPS = 8;

// Shared-memory carve-up (bytes). Ring first (16-byte aligned), then the small arrays.
struct BlockSmem {
  size_t ring, ys, redG, redP, totG, gam, tab, total;
  __host__ __device__ BlockSmem(int stages, size_t row_bytes, int math_warps) {
    ring = 0;
    ys = ring + (size_t)stages * BLK_B * row_bytes;
    redG = ys + (size_t)stages * BLK_B * sizeof(float);
    redP = redG + (size_t)math_warps * 32 * sizeof(float);
    totG = redP + (size_t)math_warps * BLK_B * sizeof(float);
    gam = totG + 32 * sizeof(float);
    tab = gam + 16 * sizeof(float);
    total = tab + 3 * 16 * sizeof(float);
  }
};

template <typename XT, int R, int LOSS>
__global__ void __launch_bounds__(32 + 32 * BLK_MAX_MATH_WARPS, 1) chain_block_kernel(const BlockParams bp) {
  constexpr int V = XVec<XT>::V;   // columns per 16-byte chunk
  constexpr int QV = V / 4;        // quads per chunk
  constexpr int B = BLK_B;
  extern __shared__ __align__(16) unsigned char smem[];
  const ChainParams& p = bp.c;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int math_warps = (blockDim.x >> 5) - 1;
  const int TM = math_warps * 32;
  const int S = bp.stages;
  const int j = p.order[blockIdx.x];
  const long long n_run = p.n_steps[j];
  const long long d = p.d;
  const size_t row_bytes = (size_t)d * sizeof(XT);  // bytes of a row that are staged
  const size_t ld_bytes = (size_t)p.ld * sizeof(XT);
  const BlockSmem L(S, row_bytes, math_warps);
  unsigned char* ring = smem + L.ring;
  float* ys = (float*)(smem + L.ys);
  float* redG = (float*)(smem + L.redG);
  float* redP = (float*)(smem + L.redP);
  float* totG = (float*)(smem + L.totG);
  float* gam = (float*)(smem + L.gam);   // gamma_0..7, [8] = 1 - a^nv
  float* tab = (float*)(smem + L.tab);   // [0..8] a^k, [16..24] eta / a^{k+1}, [32..40] 1 - a^k
  const char* shard = (const char*)p.X + (size_t)p.shard_off[j] * ld_bytes;
  const float* yshard = p.y + p.shard_off[j];
  const uint32_t* idx = p.idx + p.idx_off[j];  // padded to a multiple of B entries, all valid rows
  const long long nb = (n_run + B - 1) / B;

  if (threadIdx.x <= B) {  // power tables in fp64, rounded once
    const double a = 1.0 - bp.eta_lambda;
    double pw = 1.0;
    for (int k = 0; k < (int)threadIdx.x; ++k) pw *= a;
    tab[threadIdx.x] = (float)pw;
    tab[16 + threadIdx.x] = (float)((double)p.eta0 / (pw * a));
    tab[32 + threadIdx.x] = (float)(1.0 - pw);
  }

  if (warp == 0) {
    // =========================== serial warp ===========================================================
    const int n = lane & (B - 1);  // sample of the block this lane stands for (lanes >= B mirror, unused)
    // label prefetch: lane n < B copies y of sample n of blocks 0..S-1
    for (int s = 0; s < S; ++s) {
      if (lane < B && s < nb) cp_async4(&ys[s * B + lane], yshard + idx[(long long)s * B + lane]);
      cp_async_commit();
    }
    __syncthreads();  // tables visible (pairs with the math warps' first barrier)
    const float apow_n = tab[n], cfac_n = tab[16 + n];
    for (long long b = 0; b < nb; ++b) {
      const int nv = (int)((n_run - b * B) < (long long)B ? (n_run - b * B) : (long long)B);
      // totals of G_b (partials were written by the math warps before the previous barrier 2)
      float g_tot = 0.0f;
      for (int w = 0; w < math_warps; ++w) g_tot += redG[w * 32 + lane];
      totG[lane] = g_tot;
      __syncwarp();
      float gcol[B];  // gcol[m] = G[m][n] for m < n
#pragma unroll
      for (int m = 0; m < B; ++m) gcol[m] = (m < n) ? totG[n * (n - 1) / 2 + m] : 0.0f;
      cp_async_wait(S - 1 < 3 ? S - 1 : 3);  // this lane's label of block b has landed
      const float yn = ys[(int)(b % S) * B + n];
      __syncthreads();  // barrier 1: p_b partials are in redP
      float zacc = 0.0f;
      for (int w = 0; w < math_warps; ++w) zacc += redP[w * B + n];
      const float c_n = (n < nv) ? cfac_n : 0.0f;  // samples beyond the chain's end take no step
      float g_own = 0.0f;
#pragma unroll
      for (int m = 0; m < B; ++m) {
        const float z = apow_n * zacc;
        const float g = loss_derivative_fast<LOSS>(yn, z);
        if (m == n) g_own = g;
        const float beta_m = __shfl_sync(0xffffffffu, c_n * g, m);
        zacc = fmaf(-beta_m, gcol[m], zacc);
      }
      // gamma_n = eta g_n a^{nv-1-n}; tab[16+k] = eta / a^{k+1}, so use eta0 * a^{nv-1-n} directly
      if (lane < B) gam[lane] = (lane < nv) ? p.eta0 * g_own * tab[nv - 1 - lane] : 0.0f;
      if (lane == B) gam[B] = tab[32 + nv];
      __syncthreads();  // barrier 2: gamma published
      if (lane < B && b + S < nb) cp_async4(&ys[(int)(b % S) * B + lane], yshard + idx[(b + S) * B + lane]);
      cp_async_commit();
    }
    return;
  }

  // ============================= math warps ==============================================================
  const int tm = threadIdx.x - 32;
  bool act[R];
  float w[R][V];
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const long long c0 = ((long long)r * TM + tm) * V;
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

  // issue the copies of this thread's chunks of block blk into its ring stage
  auto prefetch_block = [&](long long blk) {
    if (blk < nb) {
      unsigned char* stage = ring + (size_t)(blk % S) * B * row_bytes;
      const uint32_t* ib = idx + blk * B;
#pragma unroll
      for (int m = 0; m < B; ++m) {
        const char* row = shard + (size_t)ib[m] * ld_bytes;
#pragma unroll
        for (int r = 0; r < R; ++r)
          if (act[r]) cp_async16(stage + (size_t)m * row_bytes + ((size_t)r * TM + tm) * 16, row + ((size_t)r * TM + tm) * 16);
      }
    }
    cp_async_commit();
  };
  // G partials of block blk -> redG (each warp its own 32 slots)
  auto gram_block = [&](long long blk) {
    float acc[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) acc[i] = 0.0f;
    if (blk < nb) {
      const unsigned char* stage = ring + (size_t)(blk % S) * B * row_bytes;
#pragma unroll
      for (int r = 0; r < R; ++r) {
        if (!act[r]) continue;
        uint4 raw[B];
#pragma unroll
        for (int m = 0; m < B; ++m)
          raw[m] = *(const uint4*)(stage + (size_t)m * row_bytes + ((size_t)r * TM + tm) * 16);
#pragma unroll
        for (int q = 0; q < QV; ++q) {
          float x[B][4];
#pragma unroll
          for (int m = 0; m < B; ++m) widen_quad<XT>(raw[m], q, x[m]);
#pragma unroll
          for (int n2 = 1; n2 < B; ++n2)
#pragma unroll
            for (int m = 0; m < n2; ++m)
#pragma unroll
              for (int e = 0; e < 4; ++e) acc[n2 * (n2 - 1) / 2 + m] = fmaf(x[m][e], x[n2][e], acc[n2 * (n2 - 1) / 2 + m]);
        }
      }
    }
    const float tot = warp_transpose_sum32(acc);
    redG[(warp - 1) * 32 + lane] = tot;
  };

  for (int s = 0; s < S; ++s) prefetch_block(s);
  cp_async_wait(S - 1 < 3 ? S - 1 : 3);  // block 0 has landed
  gram_block(0);
  __syncthreads();  // tables visible; G_0 partials visible to the serial warp

  for (long long b = 0; b < nb; ++b) {
    const unsigned char* stage = ring + (size_t)(b % S) * B * row_bytes;
    // ---- p_b = X_b w ---------------------------------------------------------------------------------
    float accp[B];
#pragma unroll
    for (int m = 0; m < B; ++m) accp[m] = 0.0f;
#pragma unroll
    for (int r = 0; r < R; ++r) {
      if (!act[r]) continue;
#pragma unroll
      for (int m = 0; m < B; ++m) {
        const uint4 raw = *(const uint4*)(stage + (size_t)m * row_bytes + ((size_t)r * TM + tm) * 16);
#pragma unroll
        for (int q = 0; q < QV; ++q) {
          float x[4];
          widen_quad<XT>(raw, q, x);
#pragma unroll
          for (int e = 0; e < 4; ++e) accp[m] = fmaf(w[r][q * 4 + e], x[e], accp[m]);
        }
      }
    }
    const float ptot = warp_transpose_sum8(accp);
    if ((lane & 3) == 0) redP[(warp - 1) * B + (lane >> 2)] = ptot;
    __syncthreads();  // barrier 1
    // ---- G_{b+1}, off the serial path -----------------------------------------------------------------
    cp_async_wait(S - 2 < 3 ? S - 2 : 3);  // block b+1 has landed
    gram_block(b + 1);
    __syncthreads();  // barrier 2: gamma_b is in gam
    // ---- w <- w - (1 - a^nv) w - sum_m gamma_m x_m -------------------------------------------------------
    float gm[B];
#pragma unroll
    for (int m = 0; m < B; ++m) gm[m] = gam[m];
    const float dl = gam[B];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      if (!act[r]) continue;
#pragma unroll
      for (int v = 0; v < V; ++v) w[r][v] = fmaf(-dl, w[r][v], w[r][v]);
#pragma unroll
      for (int m = 0; m < B; ++m) {
        const uint4 raw = *(const uint4*)(stage + (size_t)m * row_bytes + ((size_t)r * TM + tm) * 16);
#pragma unroll
        for (int q = 0; q < QV; ++q) {
          float x[4];
          widen_quad<XT>(raw, q, x);
#pragma unroll
          for (int e = 0; e < 4; ++e) w[r][q * 4 + e] = fmaf(-gm[m], x[e], w[r][q * 4 + e]);
        }
      }
    }
    prefetch_block(b + S);  // the stage of block b is free again
  }
  cp_async_wait(0);

#pragma unroll
  for (int r = 0; r < R; ++r) {
    const long long c0 = ((long long)r * TM + tm) * V;
    if (act[r]) {
      float* dst = p.W + (size_t)j * d + c0;
#pragma unroll
      for (int v = 0; v < V; ++v) dst[v] = w[r][v];
    }
  }
}

}  // namespace wpsgd
