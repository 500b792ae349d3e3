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
  size_t ring, redG, redP, totG, gam, tab, total;
  __host__ __device__ BlockSmem(int stages, size_t row_bytes, int math_warps) {
    ring = 0;
    redG = ring + (size_t)stages * BLK_B * row_bytes;
    (void)math_warps;  // the partial-sum arrays always have room for the maximum number of math warps
    redP = redG + (size_t)BLK_MAX_MATH_WARPS * 32 * sizeof(float);
    totG = redP + (size_t)BLK_MAX_MATH_WARPS * BLK_B * sizeof(float);
    gam = totG + 32 * sizeof(float);
    tab = gam + 16 * sizeof(float);
    total = tab + 3 * 16 * sizeof(float);
  }
};

template <typename XT, int R, int LOSS, bool OVERLAP>
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
  float* redG = (float*)(smem + L.redG);   // [math warp][32] partial Gram entries
  float* redP = (float*)(smem + L.redP);   // [math warp][8] partial p
  float* totG = (float*)(smem + L.totG);   // [32] Gram entries summed over the math warps
  float* gam = (float*)(smem + L.gam);     // gamma_0..7, [8] = 1 - a^nv
  float* tab = (float*)(smem + L.tab);     // [0..8] a^k, [16..24] eta / a^{k+1}, [32..40] 1 - a^k
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
    // Every lane runs the whole B-step recurrence redundantly on its own copy of the block's scalars (no
    // shuffle inside the dependent chain); lanes only differ in which partial sums they add up and in
    // which gamma they store. Lane n & 7 looks after the label of sample n.
    const int n = lane & (B - 1);
    for (int i = lane; i < BLK_MAX_MATH_WARPS * 32; i += 32)  // unused partial-sum slots read as zero
      if (i >= math_warps * 32) redG[i] = 0.0f;
    for (int i = lane; i < BLK_MAX_MATH_WARPS * B; i += 32)
      if (i >= math_warps * B) redP[i] = 0.0f;
    // label pipeline in registers: label of block b+1 and sample id of block b+2 are in flight during block b
    float y_nxt = 0.0f;
    uint32_t id_nxt = 0u;
    if (nb > 0) y_nxt = yshard[idx[n]];
    if (nb > 1) id_nxt = idx[B + n];
    __syncthreads();  // tables visible (pairs with the math warps' first barrier)
    float apw[B], cfac[B];
#pragma unroll
    for (int m = 0; m < B; ++m) { apw[m] = tab[m]; cfac[m] = tab[16 + m]; }

    for (long long b = 0; b < nb; ++b) {
      const int nv = (int)((n_run - b * B) < (long long)B ? (n_run - b * B) : (long long)B);
      const float y_cur = y_nxt;
      if (b + 1 < nb) y_nxt = yshard[id_nxt];
      if (b + 2 < nb) id_nxt = idx[(b + 2) * B + n];
      const float a_nv = tab[nv], dl_nv = tab[32 + nv];
      // per-sample constants with everything folded in that does not depend on the chain:
      // t_n = sc_n (p_n - sum_m beta_m G_mn) is the argument of the loss derivative, beta_n = cf_n * f(t_n)
      float yv[B], sc[B], cf[B];
#pragma unroll
      for (int m = 0; m < B; ++m) {
        yv[m] = __shfl_sync(0xffffffffu, y_cur, m);
        if (LOSS == LOSS_LOGISTIC) {  // g = -y / (1 + 2^t), t = y a^n log2(e) (...)
          sc[m] = yv[m] * apw[m] * 1.4426950408889634f;
          cf[m] = -yv[m] * cfac[m];
        } else if (LOSS == LOSS_HINGE) {  // g = -y if t < 1, t = y a^n (...)
          sc[m] = yv[m] * apw[m];
          cf[m] = -yv[m] * cfac[m];
        } else {  // g = t - y, t = a^n (...)
          sc[m] = apw[m];
          cf[m] = cfac[m];
        }
        if (m >= nv) cf[m] = 0.0f;  // samples beyond the chain's end take no step
      }
      float Gs[BLK_PAIRS];  // sc_n G_mn at [n(n-1)/2 + m], m < n
      auto gather_gram = [&]() {
        float gp[BLK_MAX_MATH_WARPS];
#pragma unroll
        for (int w = 0; w < BLK_MAX_MATH_WARPS; ++w) gp[w] = redG[w * 32 + lane];
        totG[lane] = ((gp[0] + gp[1]) + (gp[2] + gp[3])) + ((gp[4] + gp[5]) + (gp[6] + gp[7]));
        __syncwarp();
#pragma unroll
        for (int i = 0; i < BLK_PAIRS / 4; ++i) {
          const float4 q = ((const float4*)totG)[i];
          Gs[4 * i] = q.x; Gs[4 * i + 1] = q.y; Gs[4 * i + 2] = q.z; Gs[4 * i + 3] = q.w;
        }
        __syncwarp();
#pragma unroll
        for (int n2 = 1; n2 < B; ++n2)
#pragma unroll
          for (int m = 0; m < n2; ++m) Gs[n2 * (n2 - 1) / 2 + m] *= sc[n2];
      };
      if (OVERLAP) gather_gram();  // G_b was finished by the math warps during the previous block
      __syncthreads();             // barrier 1: p_b partials (and, without overlap, G_b partials) are in place
      if (!OVERLAP) gather_gram();
      float pp[BLK_MAX_MATH_WARPS];
#pragma unroll
      for (int w = 0; w < BLK_MAX_MATH_WARPS; ++w) pp[w] = redP[w * B + n];
      const float psum = ((pp[0] + pp[1]) + (pp[2] + pp[3])) + ((pp[4] + pp[5]) + (pp[6] + pp[7]));
      float t[B], beta[B];
#pragma unroll
      for (int m = 0; m < B; ++m) t[m] = sc[m] * __shfl_sync(0xffffffffu, psum, m);
#pragma unroll
      for (int m = 0; m < B; ++m) {
        if (LOSS == LOSS_LOGISTIC) {
          float e, r;
          asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(t[m]));
          asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(1.0f + e));
          beta[m] = cf[m] * r;
        } else if (LOSS == LOSS_HINGE) {
          beta[m] = (t[m] < 1.0f) ? cf[m] : 0.0f;
        } else {
          beta[m] = cf[m] * (t[m] - yv[m]);
        }
#pragma unroll
        for (int n2 = m + 1; n2 < B; ++n2) t[n2] = fmaf(-beta[m], Gs[n2 * (n2 - 1) / 2 + m], t[n2]);
      }
      // gamma_m = eta g_m a^{nv-1-m} = beta_m a^{nv}
      float mine = dl_nv;
#pragma unroll
      for (int m = 0; m < B; ++m)
        if (lane == m) mine = beta[m] * a_nv;
      if (lane <= B) gam[lane] = mine;
      __syncthreads();  // barrier 2: gamma published
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

  // sample ids of a block: 8 consecutive entries, 32-byte aligned (every node's stream starts on a multiple of 8)
  auto load_ids = [&](long long blk, uint4& lo, uint4& hi) {
    if (blk < nb) {
      const uint4* q = (const uint4*)(idx + blk * B);
      lo = __ldg(q);
      hi = __ldg(q + 1);
    }
  };
  // issue the copies of this thread's chunks of block blk into ring stage stg (one commit group per call)
  auto prefetch_block = [&](long long blk, int stg, const uint4& i_lo, const uint4& i_hi) {
    if (blk < nb) {
      unsigned char* stage = ring + (size_t)stg * B * row_bytes;
      const uint32_t ib[B] = {i_lo.x, i_lo.y, i_lo.z, i_lo.w, i_hi.x, i_hi.y, i_hi.z, i_hi.w};
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
  // this thread's chunks of the 8 rows of a landed block, shared memory -> registers (the only read of them)
  auto load_raw = [&](int stg, uint4 (&raw)[R][B]) {
    const unsigned char* stage = ring + (size_t)stg * B * row_bytes;
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
      for (int m = 0; m < B; ++m)
        raw[r][m] = act[r] ? *(const uint4*)(stage + (size_t)m * row_bytes + ((size_t)r * TM + tm) * 16)
                           : make_uint4(0u, 0u, 0u, 0u);
  };
  // Gram partials (and, when WITH_P, p partials against the current model) of the block held in raw
  auto products = [&](const uint4 (&raw)[R][B], float (&acc)[32], float (&accp)[B], bool with_g, bool with_p) {
#pragma unroll
    for (int r = 0; r < R; ++r) {
#pragma unroll
      for (int q = 0; q < QV; ++q) {
        float x[B][4];
#pragma unroll
        for (int m = 0; m < B; ++m) widen_quad<XT>(raw[r][m], q, x[m]);
        if (with_g) {
#pragma unroll
          for (int n2 = 1; n2 < B; ++n2)
#pragma unroll
            for (int m = 0; m < n2; ++m)
#pragma unroll
              for (int e = 0; e < 4; ++e)
                acc[n2 * (n2 - 1) / 2 + m] = fmaf(x[m][e], x[n2][e], acc[n2 * (n2 - 1) / 2 + m]);
        }
        if (with_p) {
#pragma unroll
          for (int m = 0; m < B; ++m)
#pragma unroll
            for (int e = 0; e < 4; ++e) accp[m] = fmaf(w[r][q * 4 + e], x[m][e], accp[m]);
        }
      }
    }
  };
  auto publish_g = [&](float (&acc)[32]) {
    const float tot = warp_transpose_sum32(acc);
    redG[(warp - 1) * 32 + lane] = tot;
  };
  auto publish_p = [&](float (&accp)[B]) {
    const float ptot = warp_transpose_sum8(accp);
    if ((lane & 3) == 0) redP[(warp - 1) * B + (lane >> 2)] = ptot;
  };
  // w <- w - (1 - a^nv) w - sum_m gamma_m x_m with the rows held in raw
  auto update = [&](const uint4 (&raw)[R][B]) {
    float gm[B];
#pragma unroll
    for (int m = 0; m < B; ++m) gm[m] = gam[m];
    const float dl = gam[B];
#pragma unroll
    for (int r = 0; r < R; ++r) {
#pragma unroll
      for (int v = 0; v < V; ++v) w[r][v] = fmaf(-dl, w[r][v], w[r][v]);
#pragma unroll
      for (int m = 0; m < B; ++m)
#pragma unroll
        for (int q = 0; q < QV; ++q) {
          float x[4];
          widen_quad<XT>(raw[r][m], q, x);
#pragma unroll
          for (int e = 0; e < 4; ++e) w[r][q * 4 + e] = fmaf(-gm[m], x[e], w[r][q * 4 + e]);
        }
    }
  };

  uint4 id_lo = make_uint4(0, 0, 0, 0), id_hi = make_uint4(0, 0, 0, 0);
  for (int s = 0; s < S; ++s) {
    load_ids(s, id_lo, id_hi);
    prefetch_block(s, s, id_lo, id_hi);
  }
  load_ids(S, id_lo, id_hi);
  float acc[32], accp[B];

  if (OVERLAP) {
    // Two register copies of row blocks: `cur` (block b: p_b, update) and `nxt` (block b+1: G_{b+1}).
    uint4 cur[R][B], nxt[R][B];
    cp_async_wait(S - 1 < 3 ? S - 1 : 3);  // block 0 has landed
    load_raw(0, cur);
    prefetch_block(S, 0, id_lo, id_hi);    // its stage is free again at once
    load_ids(S + 1, id_lo, id_hi);
#pragma unroll
    for (int i = 0; i < 32; ++i) acc[i] = 0.0f;
    products(cur, acc, accp, true, false);
    publish_g(acc);
    __syncthreads();  // tables visible; G_0 partials visible to the serial warp
    int st = (S > 1) ? 1 : 0;  // ring stage of block b+1
    for (long long b = 0; b < nb; ++b) {
#pragma unroll
      for (int m = 0; m < B; ++m) accp[m] = 0.0f;
      products(cur, acc, accp, false, true);  // p_b = X_b w
      publish_p(accp);
      __syncthreads();  // barrier 1
      // G_{b+1}, off the serial path
#pragma unroll
      for (int i = 0; i < 32; ++i) acc[i] = 0.0f;
      if (b + 1 < nb) {
        // groups committed so far: S + 1 + b (blocks 0 .. S+b); block b+1 must be complete
        cp_async_wait(S - 1 < 3 ? S - 1 : 3);
        load_raw(st, nxt);
        products(nxt, acc, accp, true, false);
      }
      prefetch_block(b + 1 + S, st, id_lo, id_hi);
      load_ids(b + 2 + S, id_lo, id_hi);
      publish_g(acc);
      __syncthreads();  // barrier 2: gamma_b is in gam
      update(cur);
#pragma unroll
      for (int r = 0; r < R; ++r)
#pragma unroll
        for (int m = 0; m < B; ++m) cur[r][m] = nxt[r][m];
      st = (st + 1 == S) ? 0 : st + 1;
    }
  } else {
    // One register copy: the block is read once, G_b and p_b are formed in the same pass over it, and the
    // rows stay in registers across the serial phase for the update.
    uint4 cur[R][B];
    __syncthreads();  // tables visible
    int st = 0;       // ring stage of block b
    for (long long b = 0; b < nb; ++b) {
      // groups committed so far: S + b (blocks 0 .. S+b-1); block b must be complete
      cp_async_wait(S - 1 < 3 ? S - 1 : 3);
      load_raw(st, cur);
      prefetch_block(b + S, st, id_lo, id_hi);
      load_ids(b + 1 + S, id_lo, id_hi);
#pragma unroll
      for (int i = 0; i < 32; ++i) acc[i] = 0.0f;
#pragma unroll
      for (int m = 0; m < B; ++m) accp[m] = 0.0f;
      products(cur, acc, accp, true, true);
      publish_p(accp);
      publish_g(acc);
      __syncthreads();  // barrier 1
      __syncthreads();  // barrier 2: gamma_b is in gam
      update(cur);
      st = (st + 1 == S) ? 0 : st + 1;
    }
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

// ======================================================================================================
// Small d: one warp per node, several nodes per CTA. The same blocked form, with no CTA-wide barrier at
// all: the warp forms G_b and p_b in one pass over its 8 rows (each lane owns R 16-byte column chunks),
// sums them over its lanes, every lane then runs the 8-step recurrence redundantly and applies the
// update from registers. Rows arrive through a per-warp ring filled by the lanes' own asynchronous copies.
// ======================================================================================================
namespace wpsgd {

constexpr int BLKW_WARPS = 4;  // nodes per CTA

struct BlockWarpSmem {
  size_t ring, scratch, tab, total;
  __host__ __device__ BlockWarpSmem(int stages, size_t row_bytes) {
    ring = 0;
    scratch = ring + (size_t)BLKW_WARPS * stages * BLK_B * row_bytes;
    tab = scratch + (size_t)BLKW_WARPS * 48 * sizeof(float);
    total = tab + 3 * 16 * sizeof(float);
  }
};

template <typename XT, int R, int LOSS>
__global__ void __launch_bounds__(32 * BLKW_WARPS) chain_block_warp_kernel(const BlockParams bp) {
  constexpr int V = XVec<XT>::V;
  constexpr int QV = V / 4;
  constexpr int B = BLK_B;
  extern __shared__ __align__(16) unsigned char smem[];
  const ChainParams& p = bp.c;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int S = bp.stages;
  const long long d = p.d;
  const size_t row_bytes = (size_t)d * sizeof(XT);
  const size_t ld_bytes = (size_t)p.ld * sizeof(XT);
  const BlockWarpSmem L(S, row_bytes);
  unsigned char* ring = smem + L.ring + (size_t)warp * S * B * row_bytes;
  float* scratch = (float*)(smem + L.scratch) + warp * 48;  // [0..27] G entries, [32..39] p
  float* tab = (float*)(smem + L.tab);

  if (threadIdx.x <= B) {  // power tables in fp64, rounded once
    const double a = 1.0 - bp.eta_lambda;
    double pw = 1.0;
    for (int k = 0; k < (int)threadIdx.x; ++k) pw *= a;
    tab[threadIdx.x] = (float)pw;
    tab[16 + threadIdx.x] = (float)((double)p.eta0 / (pw * a));
    tab[32 + threadIdx.x] = (float)(1.0 - pw);
  }
  __syncthreads();  // the only CTA-wide barrier; every warp passes it exactly once
  const int slot = (int)blockIdx.x * BLKW_WARPS + warp;
  if (slot >= p.k) return;
  const int j = p.order[slot];
  const long long n_run = p.n_steps[j];
  const long long nb = (n_run + B - 1) / B;
  const char* shard = (const char*)p.X + (size_t)p.shard_off[j] * ld_bytes;
  const float* yshard = p.y + p.shard_off[j];
  const uint32_t* idx = p.idx + p.idx_off[j];
  const int n = lane & (B - 1);

  float apw[B], cfac[B];
#pragma unroll
  for (int m = 0; m < B; ++m) { apw[m] = tab[m]; cfac[m] = tab[16 + m]; }

  bool act[R];
  float w[R][V];
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const long long c0 = ((long long)r * 32 + lane) * V;
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

  auto load_ids = [&](long long blk, uint4& lo, uint4& hi) {
    if (blk < nb) {
      const uint4* q = (const uint4*)(idx + blk * B);
      lo = __ldg(q);
      hi = __ldg(q + 1);
    }
  };
  auto prefetch_block = [&](long long blk, int stg, const uint4& i_lo, const uint4& i_hi) {
    if (blk < nb) {
      unsigned char* stage = ring + (size_t)stg * B * row_bytes;
      const uint32_t ib[B] = {i_lo.x, i_lo.y, i_lo.z, i_lo.w, i_hi.x, i_hi.y, i_hi.z, i_hi.w};
#pragma unroll
      for (int m = 0; m < B; ++m) {
        const char* row = shard + (size_t)ib[m] * ld_bytes;
#pragma unroll
        for (int r = 0; r < R; ++r)
          if (act[r]) cp_async16(stage + (size_t)m * row_bytes + ((size_t)r * 32 + lane) * 16, row + ((size_t)r * 32 + lane) * 16);
      }
    }
    cp_async_commit();
  };

  uint4 id_lo = make_uint4(0, 0, 0, 0), id_hi = make_uint4(0, 0, 0, 0);
  for (int s = 0; s < S; ++s) {
    load_ids(s, id_lo, id_hi);
    prefetch_block(s, s, id_lo, id_hi);
  }
  load_ids(S, id_lo, id_hi);
  float y_nxt = 0.0f;
  uint32_t id_nxt = 0u;
  if (nb > 0) y_nxt = yshard[idx[n]];
  if (nb > 1) id_nxt = idx[B + n];

  int st = 0;
  for (long long b = 0; b < nb; ++b) {
    const int nv = (int)((n_run - b * B) < (long long)B ? (n_run - b * B) : (long long)B);
    const float y_cur = y_nxt;
    if (b + 1 < nb) y_nxt = yshard[id_nxt];
    if (b + 2 < nb) id_nxt = idx[(b + 2) * B + n];
    // ---- rows of block b: shared memory -> registers, then refill the stage --------------------------------
    cp_async_wait(S - 1 < 3 ? S - 1 : 3);  // groups committed: S + b; block b must be complete
    uint4 raw[R][B];
    {
      const unsigned char* stage = ring + (size_t)st * B * row_bytes;
#pragma unroll
      for (int r = 0; r < R; ++r)
#pragma unroll
        for (int m = 0; m < B; ++m)
          raw[r][m] = act[r] ? *(const uint4*)(stage + (size_t)m * row_bytes + ((size_t)r * 32 + lane) * 16)
                             : make_uint4(0u, 0u, 0u, 0u);
    }
    prefetch_block(b + S, st, id_lo, id_hi);
    load_ids(b + 1 + S, id_lo, id_hi);
    // ---- G_b and p_b in one pass -----------------------------------------------------------------------
    float acc[32], accp[B];
#pragma unroll
    for (int i = 0; i < 32; ++i) acc[i] = 0.0f;
#pragma unroll
    for (int m = 0; m < B; ++m) accp[m] = 0.0f;
#pragma unroll
    for (int r = 0; r < R; ++r) {
#pragma unroll
      for (int q = 0; q < QV; ++q) {
        float x[B][4];
#pragma unroll
        for (int m = 0; m < B; ++m) widen_quad<XT>(raw[r][m], q, x[m]);
#pragma unroll
        for (int n2 = 1; n2 < B; ++n2)
#pragma unroll
          for (int m = 0; m < n2; ++m)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[n2 * (n2 - 1) / 2 + m] = fmaf(x[m][e], x[n2][e], acc[n2 * (n2 - 1) / 2 + m]);
#pragma unroll
        for (int m = 0; m < B; ++m)
#pragma unroll
          for (int e = 0; e < 4; ++e) accp[m] = fmaf(w[r][q * 4 + e], x[m][e], accp[m]);
      }
    }
    const float ptot = warp_transpose_sum8(accp);   // every lane: total of p_{lane >> 2}
    const float gtot = warp_transpose_sum32(acc);   // lane l: total of Gram entry l
    // all 28 + 8 totals into every lane (through the warp's scratch line)
    scratch[lane] = gtot;
    if ((lane & 3) == 0) scratch[32 + (lane >> 2)] = ptot;
    __syncwarp();
    float Gs[BLK_PAIRS], pv[B];
#pragma unroll
    for (int i = 0; i < BLK_PAIRS / 4; ++i) {
      const float4 q = ((const float4*)scratch)[i];
      Gs[4 * i] = q.x; Gs[4 * i + 1] = q.y; Gs[4 * i + 2] = q.z; Gs[4 * i + 3] = q.w;
    }
    {
      const float4 q0 = ((const float4*)scratch)[8], q1 = ((const float4*)scratch)[9];
      pv[0] = q0.x; pv[1] = q0.y; pv[2] = q0.z; pv[3] = q0.w; pv[4] = q1.x; pv[5] = q1.y; pv[6] = q1.z; pv[7] = q1.w;
    }
    __syncwarp();
    // ---- 8-step recurrence, every lane the same ----------------------------------------------------------
    const float a_nv = tab[nv], dl = tab[32 + nv];
    float t[B], beta[B], yv[B], cf[B];
#pragma unroll
    for (int m = 0; m < B; ++m) {
      yv[m] = __shfl_sync(0xffffffffu, y_cur, m);
      float sc;
      if (LOSS == LOSS_LOGISTIC) { sc = yv[m] * apw[m] * 1.4426950408889634f; cf[m] = -yv[m] * cfac[m]; }
      else if (LOSS == LOSS_HINGE) { sc = yv[m] * apw[m]; cf[m] = -yv[m] * cfac[m]; }
      else { sc = apw[m]; cf[m] = cfac[m]; }
      if (m >= nv) cf[m] = 0.0f;
      t[m] = sc * pv[m];
#pragma unroll
      for (int k2 = 0; k2 < m; ++k2) Gs[m * (m - 1) / 2 + k2] *= sc;
    }
#pragma unroll
    for (int m = 0; m < B; ++m) {
      if (LOSS == LOSS_LOGISTIC) {
        float e, r;
        asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(t[m]));
        asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(1.0f + e));
        beta[m] = cf[m] * r;
      } else if (LOSS == LOSS_HINGE) {
        beta[m] = (t[m] < 1.0f) ? cf[m] : 0.0f;
      } else {
        beta[m] = cf[m] * (t[m] - yv[m]);
      }
#pragma unroll
      for (int n2 = m + 1; n2 < B; ++n2) t[n2] = fmaf(-beta[m], Gs[n2 * (n2 - 1) / 2 + m], t[n2]);
    }
    // ---- w <- w - (1 - a^nv) w - sum_m gamma_m x_m,  gamma_m = beta_m a^nv ----------------------------------
#pragma unroll
    for (int r = 0; r < R; ++r) {
#pragma unroll
      for (int v = 0; v < V; ++v) w[r][v] = fmaf(-dl, w[r][v], w[r][v]);
#pragma unroll
      for (int m = 0; m < B; ++m) {
        const float gm = beta[m] * a_nv;
#pragma unroll
        for (int q = 0; q < QV; ++q) {
          float x[4];
          widen_quad<XT>(raw[r][m], q, x);
#pragma unroll
          for (int e = 0; e < 4; ++e) w[r][q * 4 + e] = fmaf(-gm, x[e], w[r][q * 4 + e]);
        }
      }
    }
    st = (st + 1 == S) ? 0 : st + 1;
  }
  cp_async_wait(0);

#pragma unroll
  for (int r = 0; r < R; ++r) {
    const long long c0 = ((long long)r * 32 + lane) * V;
    if (act[r]) {
      float* dst = p.W + (size_t)j * d + c0;
#pragma unroll
      for (int v = 0; v < V; ++v) dst[v] = w[r][v];
    }
  }
}

}  // namespace wpsgd
