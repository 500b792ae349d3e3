// Per-node SGD chains on dense rows, blocked form (constant step size, or eta0 / sqrt(n) with per-block tables).
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
// One CTA per node: warp 0 is the "recurrence warp" (sums the partial products, runs the B-step recurrence,
// publishes gamma); warp 1 is the "copy warp" (requests the 8 rows of a future block as bulk asynchronous
// copies, cp.async.bulk, that complete on a shared-memory barrier of the ring stage; never multicast); the other
// warps are "math warps", each thread owning fixed columns of the model in registers for the whole chain.
// A landed block is read from shared memory exactly once, into registers. Every wait on a stage barrier is
// bounded: when it runs out the kernel records a timeout in the status word, all warps leave the loop at the
// same barrier, the copy warp waits (bounded again) for copies still in flight, and the kernel returns.
//
// Per block b (overlapped schedule, one 16-byte chunk per thread):
//                math warps                               recurrence warp
//                p_b partials (needs w)  -> smem          sum G_b partials (written last round)
//                ------------------------- barrier 1 --------------------------------------
//                G_{b+1} partials -> smem                 sum p_b, B-step recurrence, gamma -> smem
//                ------------------------- barrier 2 --------------------------------------
//                w <- w - (1-a^B) w - sum gamma_m x_m     labels and constants of block b+1
// With two chunks per thread (wide rows) registers hold one block only: G_b and p_b are formed in one pass
// before barrier 1 and the math warps idle during the recurrence.
#pragma once

#include "chain_dense.cuh"
#include "common.cuh"

namespace wpsgd {

struct BlockParams {
  ChainParams c;
  int stages;            // S: blocks in the shared-memory ring (>= 2)
  double eta_lambda;     // eta * lambda in fp64
  long long spin_limit;  // polls after which a wait on arriving rows gives up
  long long drop_block;  // test hook: the rows of this block are never requested (-1: none)
  const int* group_order;  // warp-per-node kernel: node of every (CTA, warp) slot, -1 = none
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
// wait until at most `pending` of this thread's committed groups are still in flight (pending in 0..6)
__device__ __forceinline__ void cp_async_wait(int pending) {
  switch (pending) {
    case 0: asm volatile("cp.async.wait_group 0;" ::: "memory"); break;
    case 1: asm volatile("cp.async.wait_group 1;" ::: "memory"); break;
    case 2: asm volatile("cp.async.wait_group 2;" ::: "memory"); break;
    case 3: asm volatile("cp.async.wait_group 3;" ::: "memory"); break;
    case 4: asm volatile("cp.async.wait_group 4;" ::: "memory"); break;
    case 5: asm volatile("cp.async.wait_group 5;" ::: "memory"); break;
    default: asm volatile("cp.async.wait_group 6;" ::: "memory"); break;
  }
}

// ---- bulk asynchronous copies (TMA, untiled form) completing on a shared-memory barrier ------------------------
__device__ __forceinline__ void mbar_init(unsigned long long* bar, int count) {
  const uint32_t a = (uint32_t)__cvta_generic_to_shared(bar);
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(a), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive_expect_tx(unsigned long long* bar, uint32_t bytes) {
  const uint32_t a = (uint32_t)__cvta_generic_to_shared(bar);
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(a), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned long long* bar, uint32_t parity) {
  const uint32_t a = (uint32_t)__cvta_generic_to_shared(bar);
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(a), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait for the phase with the given parity to complete; false when the limit ran out.
__device__ __forceinline__ bool mbar_wait_bounded(unsigned long long* bar, uint32_t parity, long long limit) {
  for (long long i = 0; i < limit; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
// One contiguous global -> shared copy (no multicast); bytes a multiple of 16, both addresses 16-byte aligned.
__device__ __forceinline__ void bulk_copy_g2s(void* smem_dst, const void* gmem_src, uint32_t bytes, unsigned long long* bar) {
  const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst), b = (uint32_t)__cvta_generic_to_shared(bar);
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(d),
               "l"(gmem_src), "r"(bytes), "r"(b)
               : "memory");
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

// The columns of a 16-byte chunk as pairs of fp32 (the operand form of the packed FMA).
template <typename XT>
struct XPairs;
template <>
struct XPairs<float> {
  static constexpr int NP = 2;
  __device__ __forceinline__ static float2 get(const uint4& raw, int i) {
    return i == 0 ? make_float2(__uint_as_float(raw.x), __uint_as_float(raw.y))
                  : make_float2(__uint_as_float(raw.z), __uint_as_float(raw.w));
  }
};
template <>
struct XPairs<__nv_bfloat16> {
  static constexpr int NP = 4;
  __device__ __forceinline__ static float2 get(const uint4& raw, int i) {
    const uint32_t u = i == 0 ? raw.x : (i == 1 ? raw.y : (i == 2 ? raw.z : raw.w));
    return make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xffff0000u));
  }
};

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

// Logistic loss in the blocked recurrence. With t the margin times y log2(e), the step needs s(t) = 1 / (1 + 2^t):
// two special-function evaluations in the dependent chain of every sample. Inside a block the argument of sample n is
// t0_n + delta_n, where t0_n (from p_n) is known before the recurrence starts and delta_n collects the block's earlier
// steps. s and its first three derivatives at t0_n are formed for all samples of the block at once; the chain then
// only evaluates a cubic in delta_n. Remainder: |d4s/dt4| delta^4 / 24 < 2e-8 for |delta| < 1/16; a block in which
// some delta is larger is run again with the direct evaluation (kept out of the fast loop, so that no
// special-function unit sits in its dependent chain).
constexpr float LOGISTIC_DELTA_MAX = 0.0625f;
__device__ __forceinline__ float logistic_factor(float t) {
  float e, r;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(t));
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(1.0f + e));
  return r;
}
// (s, ds/dt, d2s/dt2 / 2, d3s/dt3 / 6) at t0. With x = t ln2 and f = 1/(1+e^x): df = -f(1-f), d2f = f(1-f)(1-2f),
// d3f = f(1-f)(6f(1-f) - 1).
__device__ __forceinline__ float4 logistic_jet(float t0) {
  constexpr float q = 0.6931471805599453f;
  const float f = logistic_factor(t0);
  const float h = f * (1.0f - f);
  float4 j;
  j.x = f;
  j.y = -q * h;
  j.z = (0.5f * q * q) * h * fmaf(-2.0f, f, 1.0f);
  j.w = (q * q * q / 6.0f) * h * fmaf(6.0f, h, -1.0f);
  return j;
}
// The cubic at delta (valid while |delta| < LOGISTIC_DELTA_MAX).
__device__ __forceinline__ float logistic_factor_near(const float4& jet, float delta) {
  return fmaf(delta, fmaf(delta, fmaf(delta, jet.w, jet.z), jet.y), jet.x);
}

// 8x8 b16 tiles from shared memory, four at a time (lanes 8i..8i+7 give the row addresses of tile i); each
// lane receives, per tile, the pair of elements (row = lane / 4, columns 2 (lane % 4), +1).
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const void* smem_ptr) {
  const uint32_t a = (uint32_t)__cvta_generic_to_shared(smem_ptr);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(a)
               : "memory");
}
// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col). bf16 products are exact in fp32.
__device__ __forceinline__ void mma_bf16_m16n8k16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                                  uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

constexpr int BLK_B = 8;                           // samples per block
constexpr int BLK_PAIRS = BLK_B * (BLK_B - 1) / 2;  // 28 Gram entries below the diagonal
constexpr int BLK_MAX_MATH_WARPS = 16;

// Tables of a block for the decaying schedule eta_n = eta0 / sqrt(n). With a_s = 1 - eta_s lambda and A_m the product
// of a_s over the block's first m steps: apw[m] = A_m, cfac[m] = eta_m / A_{m+1}, a_nv = A_nv, dl_nv = 1 - A_nv, and
// apw_own = A of the sample this lane looks after (lane mod B). n0 = steps the chain has run before the block. Formed
// in fp64 by the lanes of the calling warp and rounded once; all lanes of the warp must call it. (For a constant step
// size these are powers of a = 1 - eta lambda, kept in shared memory.) The blocked algebra itself does not change:
// w after n samples = A_n (w_0 - sum_{m<n} beta_m x_m) with beta_m = eta_m g_m / A_{m+1}.
template <int B>
__device__ __forceinline__ void decaying_block_tables(double eta0, double lam, long long n0, int nv, float (&apw)[B],
                                                      float (&cfac)[B], float& apw_own, float& a_nv, float& dl_nv) {
  const int m = (int)(threadIdx.x & (B - 1));
  // 1 / sqrt(n) and 1 / A from the fp32 special-function unit plus one Newton step in fp64 (relative error below
  // 1e-12): no fp64 square root or division on the way
  const double nn = (double)(n0 + m + 1);
  double rs = (double)rsqrtf((float)nn);
  rs = rs * fma(-0.5 * nn, rs * rs, 1.5);
  const double eta = eta0 * rs;
  double ia = fma(-eta, lam, 1.0);  // becomes A_{m+1}: inclusive product over the block's steps 0..m
#pragma unroll
  for (int o = 1; o < B; o <<= 1) {
    const double v = __shfl_up_sync(0xffffffffu, ia, o, B);
    if (m >= o) ia *= v;
  }
  double ea = __shfl_up_sync(0xffffffffu, ia, 1, B);  // A_m
  if (m == 0) ea = 1.0;
  double rc = (double)__frcp_rn((float)ia);
  rc = rc * fma(-ia, rc, 2.0);
  const float apw_f = (float)ea, cf_f = (float)(eta * rc);
#pragma unroll
  for (int q = 0; q < B; ++q) {
    apw[q] = __shfl_sync(0xffffffffu, apw_f, q, B);
    cfac[q] = __shfl_sync(0xffffffffu, cf_f, q, B);
  }
  const double a_end = nv > 0 ? __shfl_sync(0xffffffffu, ia, nv - 1, B) : 1.0;
  apw_own = apw_f;
  a_nv = (float)a_end;
  dl_nv = (float)(1.0 - a_end);
}

// Per-sample constants of a block of 8 with everything folded in that does not depend on the chain:
// t_n = sc_n (p_n - sum_m beta_m G_mn) is the argument of the loss derivative, beta_n = cf_n * f(t_n).
// apw[m] = a^m, cfac[m] = eta / a^{m+1}; samples from nv on lie beyond the chain's end and take no step.
template <int LOSS>
__device__ __forceinline__ void block8_constants(const float (&yv)[BLK_B], const float (&apw)[BLK_B], const float (&cfac)[BLK_B],
                                                 int nv, float (&sc)[BLK_B], float (&cf)[BLK_B]) {
#pragma unroll
  for (int m = 0; m < BLK_B; ++m) {
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
    if (m >= nv) cf[m] = 0.0f;
  }
}

// The 8-step scalar recurrence of a block, every lane the same (no shuffle in the dependent chain). On entry
// t[n] = sc_n p_n and Gs[n (n - 1) / 2 + m] = sc_n G_mn (m < n); on exit beta[m] = eta g_m / a^{m+1}. For the logistic
// loss jets_smem (8 float4 of the warp's own) receives the expansions of the factor around the block's margins:
// lane n < 8 expands its own sample at t_own, every lane then reads all eight; a block whose steps move a margin
// beyond the range of the cubic is run again with the direct evaluation.
template <int LOSS>
__device__ __forceinline__ void block8_recurrence(float (&t)[BLK_B], const float (&Gs)[BLK_PAIRS], const float (&cf)[BLK_B],
                                                  const float (&yv)[BLK_B], float t_own, float4* jets_smem,
                                                  float (&beta)[BLK_B]) {
  constexpr int B = BLK_B;
  if (LOSS == LOSS_LOGISTIC) {
    const int lane = threadIdx.x & 31;
    if (lane < B) jets_smem[lane] = logistic_jet(t_own);
    __syncwarp();
    float4 jet[B];
    float dlt[B];
#pragma unroll
    for (int m = 0; m < B; ++m) {
      jet[m] = jets_smem[m];
      dlt[m] = 0.0f;
    }
    float dmax = 0.0f;  // (jets_smem is written again a block later, behind at least one warp-wide barrier of the caller)
#pragma unroll
    for (int m = 0; m < B; ++m) {
      dmax = fmaxf(dmax, fabsf(dlt[m]));
      beta[m] = cf[m] * logistic_factor_near(jet[m], dlt[m]);
#pragma unroll
      for (int n2 = m + 1; n2 < B; ++n2) dlt[n2] = fmaf(-beta[m], Gs[n2 * (n2 - 1) / 2 + m], dlt[n2]);
    }
    if (!(dmax < LOGISTIC_DELTA_MAX)) {  // rare: some step of the block moved a margin far; direct evaluation
#pragma unroll 1
      for (int m = 0; m < B; ++m) {
        float tm_ = 0.0f, cfm = 0.0f;
#pragma unroll
        for (int q = 0; q < B; ++q)
          if (q == m) { tm_ = t[q]; cfm = cf[q]; }
        const float bm = cfm * logistic_factor(tm_);
#pragma unroll
        for (int q = 0; q < B; ++q)
          if (q == m) beta[q] = bm;
#pragma unroll
        for (int n2 = 1; n2 < B; ++n2)
#pragma unroll
          for (int q = 0; q < n2; ++q)
            if (q == m) t[n2] = fmaf(-bm, Gs[n2 * (n2 - 1) / 2 + q], t[n2]);
      }
    }
  } else {
#pragma unroll
    for (int m = 0; m < B; ++m) {
      if (LOSS == LOSS_HINGE) beta[m] = (t[m] < 1.0f) ? cf[m] : 0.0f;
      else beta[m] = cf[m] * (t[m] - yv[m]);
#pragma unroll
      for (int n2 = m + 1; n2 < B; ++n2) t[n2] = fmaf(-beta[m], Gs[n2 * (n2 - 1) / 2 + m], t[n2]);
    }
  }
}

// Shared-memory carve-up (bytes). Ring first (16-byte aligned), then the small arrays.
struct BlockSmem {
  size_t ring, redG, redP, totG, gam, tab, jet, bars, flag, total;
  __host__ __device__ BlockSmem(int stages, size_t row_bytes, int math_warps) {
    ring = 0;
    redG = ring + (size_t)stages * BLK_B * row_bytes;
    (void)math_warps;  // the partial-sum arrays always have room for the maximum number of math warps
    redP = redG + (size_t)BLK_MAX_MATH_WARPS * 64 * sizeof(float);
    totG = redP + (size_t)BLK_MAX_MATH_WARPS * BLK_B * sizeof(float);
    gam = totG + 64 * sizeof(float);
    tab = gam + 16 * sizeof(float);
    jet = tab + 3 * 16 * sizeof(float);  // 8 x (s, s', s''/2, s'''/6) of the logistic factor
    bars = jet + 8 * 4 * sizeof(float);  // one arrival barrier per ring stage (up to 8)
    flag = bars + 8 * sizeof(unsigned long long);
    total = flag + 16;
  }
};

template <typename XT, int R, int LOSS, bool OVERLAP, int MAXW>
__global__ void __launch_bounds__(64 + 32 * MAXW, 1) chain_block_kernel(const BlockParams bp) {
  constexpr int V = XVec<XT>::V;   // columns per 16-byte chunk
  constexpr int QV = V / 4;        // quads per chunk
  constexpr int B = BLK_B;
  extern __shared__ __align__(16) unsigned char smem[];
  const ChainParams& p = bp.c;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int math_warps = (blockDim.x >> 5) - 2;  // warp 0: recurrence, warp 1: row copies, the rest: math
  const int TM = math_warps * 32;
  const int S = bp.stages;
  const int j = p.order[blockIdx.x];
  const long long n_run = p.n_steps[j];
  const long long d = p.d;
  constexpr int GW = 32;  // Gram partials per math warp (28 used)
  const size_t row_bytes = (size_t)d * sizeof(XT) + (sizeof(XT) == 2 ? 16 : 0);  // stride of a staged row
  const size_t ld_bytes = (size_t)p.ld * sizeof(XT);
  const BlockSmem L(S, row_bytes, math_warps);
  unsigned char* ring = smem + L.ring;
  float* redG = (float*)(smem + L.redG);   // [math warp][32] partial Gram entries
  float* redP = (float*)(smem + L.redP);   // [math warp][8] partial p
  float* totG = (float*)(smem + L.totG);   // [32] Gram entries summed over the math warps
  float* gam = (float*)(smem + L.gam);     // gamma_0..7, [8] = 1 - a^nv
  float* tab = (float*)(smem + L.tab);     // [0..8] a^k, [16..24] eta / a^{k+1}, [32..40] 1 - a^k
  float4* jets = (float4*)(smem + L.jet);  // logistic factor and derivatives of the block's 8 samples
  unsigned long long* bars = (unsigned long long*)(smem + L.bars);  // bars[s]: rows of the block in stage s have landed
  volatile int* give_up = (volatile int*)(smem + L.flag);           // set when a bounded wait ran out
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
  if (threadIdx.x == 32) {
    for (int s = 0; s < S; ++s) mbar_init(&bars[s], 1);
    *give_up = 0;
    mbar_fence_init();
  }
  __syncthreads();  // tables and barriers are set up

  if (warp == 0) {
    // =========================== serial warp ===========================================================
    // Every lane runs the whole B-step recurrence redundantly on its own copy of the block's scalars (no
    // shuffle inside the dependent chain); lanes only differ in which partial sums they add up and in
    // which gamma they store. Lane n & 7 looks after the label of sample n.
    const int n = lane & (B - 1);
    for (int i = lane; i < MAXW * GW; i += 32)  // unused partial-sum slots read as zero
      if (i >= math_warps * GW) redG[i] = 0.0f;
    for (int i = lane; i < MAXW * B; i += 32)
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
    const bool decaying = p.sched == LR_INV_SQRT;
    const long long first_j = p.first ? p.first[j] : 0;

    for (long long b = 0; b < nb; ++b) {
      const int nv = (int)((n_run - b * B) < (long long)B ? (n_run - b * B) : (long long)B);
      const float y_cur = y_nxt;
      if (b + 1 < nb) y_nxt = yshard[id_nxt];
      if (b + 2 < nb) id_nxt = idx[(b + 2) * B + n];
      float a_nv = tab[nv], dl_nv = tab[32 + nv], apw_own = tab[n];
      if (decaying) decaying_block_tables<B>((double)p.eta0, (double)p.lambda, first_j + b * B, nv, apw, cfac, apw_own, a_nv, dl_nv);
      float yv[B], sc[B], cf[B];
#pragma unroll
      for (int m = 0; m < B; ++m) yv[m] = __shfl_sync(0xffffffffu, y_cur, m);
      block8_constants<LOSS>(yv, apw, cfac, nv, sc, cf);
      float Gs[BLK_PAIRS];  // sc_n G_mn at [n(n-1)/2 + m], m < n
      auto gather_gram = [&]() {
        {
          float gp[MAXW];
#pragma unroll
          for (int w = 0; w < MAXW; ++w) gp[w] = redG[w * 32 + lane];
#pragma unroll
          for (int h = MAXW / 2; h >= 1; h >>= 1)
#pragma unroll
            for (int w = 0; w < h; ++w) gp[w] += gp[w + h];
          totG[lane] = gp[0];
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
        }
      };
      if (OVERLAP) gather_gram();  // G_b was finished by the math warps during the previous block
      __syncthreads();             // barrier 1: p_b partials (and, without overlap, G_b partials) are in place
      // A wait that ran out is flagged before barrier 1 (before barrier 2 in the overlapped schedule); every warp
      // reads the flag right after that barrier and nothing writes it again before all have read it, so all
      // warps leave the loop at the same point and no barrier is left waiting.
      if (!OVERLAP && *give_up) break;
      if (!OVERLAP) gather_gram();
      float pp[MAXW];
#pragma unroll
      for (int w = 0; w < MAXW; ++w) pp[w] = redP[w * B + n];
#pragma unroll
      for (int h = MAXW / 2; h >= 1; h >>= 1)
#pragma unroll
        for (int w = 0; w < h; ++w) pp[w] += pp[w + h];
      const float psum = pp[0];
      float t[B], beta[B];
#pragma unroll
      for (int m = 0; m < B; ++m) t[m] = sc[m] * __shfl_sync(0xffffffffu, psum, m);
      block8_recurrence<LOSS>(t, Gs, cf, yv, y_cur * apw_own * 1.4426950408889634f * psum, jets, beta);
      // gamma_m = eta g_m a^{nv-1-m} = beta_m a^{nv}
      float mine = dl_nv;
#pragma unroll
      for (int m = 0; m < B; ++m)
        if (lane == m) mine = beta[m] * a_nv;
      if (lane <= B) gam[lane] = mine;
      __syncthreads();  // barrier 2: gamma published
      if (OVERLAP && *give_up) break;
    }
    return;
  }

  if (warp == 1) {
    // =========================== copy warp ==============================================================
    // Lane m < 8 requests row m of a block as one bulk copy; the eight copies complete on the stage's barrier.
    // A stage is refilled only after a CTA barrier that every reader of its previous content has passed.
    const uint32_t copy_bytes = (uint32_t)((size_t)d * sizeof(XT));
    uint32_t id_next = 0u;  // sample id of this lane's row in the next block to request
    auto peek = [&](long long blk) {
      if (lane < B && blk < nb) id_next = idx[blk * B + lane];
    };
    auto request = [&](long long blk, int stg) {
      if (blk < nb && blk != bp.drop_block) {
        if (lane == 0) mbar_arrive_expect_tx(&bars[stg], B * copy_bytes);
        __syncwarp();
        if (lane < B)
          bulk_copy_g2s(ring + ((size_t)stg * B + lane) * row_bytes, shard + (size_t)id_next * ld_bytes, copy_bytes, &bars[stg]);
      }
    };
    long long requested = 0;  // blocks 0 .. requested-1 have been asked for
    for (int s = 0; s < S; ++s) {
      peek(s);
      request(s, s);
      ++requested;
    }
    peek(requested);
    __syncthreads();  // pairs with the other warps' start-up barrier
    int st = 0;
    long long b = 0;
    if (OVERLAP) {
      // block 0 went to registers before the start-up barrier: stage 0 takes block S now
      request(requested, 0);
      ++requested;
      peek(requested);
      st = (S > 1) ? 1 : 0;
    }
    bool stop = false;
    for (; b < nb; ++b) {
      __syncthreads();  // barrier 1
      if (!OVERLAP) {
        if (*give_up) { stop = true; break; }
        request(requested, st);  // every math warp has block b in registers: its stage takes block b + S
        ++requested;
        peek(requested);
      }
      __syncthreads();  // barrier 2
      if (OVERLAP) {
        if (*give_up) { stop = true; break; }
        request(requested, st);  // block b+1 went to registers between the barriers: its stage takes block b+1+S
        ++requested;
        peek(requested);
      }
      st = (st + 1 == S) ? 0 : st + 1;
    }
    if (stop) {
      // leave no copy in flight into this CTA's shared memory: wait (bounded) on the stage of every block that
      // was requested and may not have landed yet
      long long blk = b - 1 > 0 ? b - 1 : 0;
      for (; blk < requested && blk < nb; ++blk)
        if (blk != bp.drop_block) mbar_wait_bounded(&bars[blk % S], (uint32_t)((blk / S) & 1), bp.spin_limit);
    }
    return;
  }

  // ============================= math warps ==============================================================
  const int tm = threadIdx.x - 64;
  const int mw = warp - 2;  // math warp number
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

  // wait (bounded) until the rows of block blk have landed in their stage
  auto wait_rows = [&](int stg, uint32_t parity) {
    if (!mbar_wait_bounded(&bars[stg], parity, bp.spin_limit)) {
      set_status(p.status, DEV_TIMEOUT, 1, (long long)blockIdx.x);
      *give_up = 1;
    }
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
    redG[mw * 32 + lane] = tot;
  };
  auto publish_p = [&](float (&accp)[B]) {
    const float ptot = warp_transpose_sum8(accp);
    if ((lane & 3) == 0) redP[mw * B + (lane >> 2)] = ptot;
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

  float acc[32], accp[B];

  if (OVERLAP) {
    // Two register copies of row blocks: `cur` (block b: p_b, update) and `nxt` (block b+1: G_{b+1}).
    uint4 cur[R][B], nxt[R][B];
#pragma unroll
    for (int i = 0; i < 32; ++i) acc[i] = 0.0f;
    if (nb > 0) {
      wait_rows(0, 0u);
      load_raw(0, cur);
      products(cur, acc, accp, true, false);
    }
    publish_g(acc);
    __syncthreads();  // start-up barrier: G_0 partials visible to the serial warp, stage 0 free
    int st = (S > 1) ? 1 : 0;  // ring stage of block b+1 ...
    uint32_t par = (S > 1) ? 0u : 1u;  // ... and the parity of the barrier phase that brings it
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
        wait_rows(st, par);
        load_raw(st, nxt);
        products(nxt, acc, accp, true, false);
      }
      publish_g(acc);
      __syncthreads();  // barrier 2: gamma_b is in gam; the stage of block b+1 is free
      if (*give_up) break;
      update(cur);
#pragma unroll
      for (int r = 0; r < R; ++r)
#pragma unroll
        for (int m = 0; m < B; ++m) cur[r][m] = nxt[r][m];
      if (++st == S) { st = 0; par ^= 1u; }
    }
  } else {
    // One register copy: the block is read once, G_b and p_b are formed in the same pass over it, and the
    // rows stay in registers across the serial phase for the update.
    uint4 cur[R][B];
    __syncthreads();  // start-up barrier
    int st = 0;       // ring stage of block b ...
    uint32_t par = 0u;  // ... and the parity of the barrier phase that brings it
    for (long long b = 0; b < nb; ++b) {
      wait_rows(st, par);
      load_raw(st, cur);
#pragma unroll
      for (int m = 0; m < B; ++m) accp[m] = 0.0f;
#pragma unroll
      for (int i = 0; i < 32; ++i) acc[i] = 0.0f;
      products(cur, acc, accp, true, true);
      publish_p(accp);
      publish_g(acc);
      __syncthreads();  // barrier 1: the stage of block b is free
      if (*give_up) break;
      __syncthreads();  // barrier 2: gamma_b is in gam
      update(cur);
      if (++st == S) { st = 0; par ^= 1u; }
    }
  }

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

constexpr int BLKW_MAX_WARPS = 4;  // most nodes per CTA

struct BlockWarpSmem {
  size_t ring, scratch, tab, total;
  __host__ __device__ BlockWarpSmem(int stages, size_t row_bytes, int warps) {
    ring = 0;
    scratch = ring + (size_t)warps * stages * BLK_B * row_bytes;
    tab = scratch + (size_t)warps * 72 * sizeof(float);
    total = tab + 3 * 16 * sizeof(float);
  }
};

// DECAY: the step size decays (per-block tables); the constant schedule is compiled without that code
template <typename XT, int R, int LOSS, bool DECAY>
__global__ void __launch_bounds__(32 * BLKW_MAX_WARPS) chain_block_warp_kernel(const BlockParams bp) {
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
  const int nwarps = blockDim.x >> 5;
  const BlockWarpSmem L(S, row_bytes, nwarps);
  unsigned char* ring = smem + L.ring + (size_t)warp * S * B * row_bytes;
  float* scratch = (float*)(smem + L.scratch) + warp * 72;  // [0..27] G entries, [32..39] p, [40..71] logistic expansions
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
  // slot -> node table (group_order): the nodes of a CTA are chosen on the host so that every CTA carries about
  // the same total number of steps; -1 marks an unused slot
  const int j = bp.group_order[(int)blockIdx.x * nwarps + warp];
  if (j < 0) return;
  const long long n_run = p.n_steps[j];
  const long long nb = (n_run + B - 1) / B;
  const char* shard = (const char*)p.X + (size_t)p.shard_off[j] * ld_bytes;
  const float* yshard = p.y + p.shard_off[j];
  const uint32_t* idx = p.idx + p.idx_off[j];
  const int n = lane & (B - 1);

  float apw[B], cfac[B];
#pragma unroll
  for (int m = 0; m < B; ++m) { apw[m] = tab[m]; cfac[m] = tab[16 + m]; }
  const long long first_j = (DECAY && p.first) ? p.first[j] : 0;

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
    // packed two-wide fp32 FMAs: even and odd columns accumulate side by side and are added at the end
    float acc[32], accp[B];
    {
      constexpr int NP = XPairs<XT>::NP;
      float2 acc2[BLK_PAIRS], accp2[B];
#pragma unroll
      for (int i = 0; i < BLK_PAIRS; ++i) acc2[i] = make_float2(0.0f, 0.0f);
#pragma unroll
      for (int m = 0; m < B; ++m) accp2[m] = make_float2(0.0f, 0.0f);
#pragma unroll
      for (int r = 0; r < R; ++r) {
#pragma unroll
        for (int i = 0; i < NP; ++i) {
          float2 x2[B];
#pragma unroll
          for (int m = 0; m < B; ++m) x2[m] = XPairs<XT>::get(raw[r][m], i);
#pragma unroll
          for (int n2 = 1; n2 < B; ++n2)
#pragma unroll
            for (int m = 0; m < n2; ++m) acc2[n2 * (n2 - 1) / 2 + m] = __ffma2_rn(x2[m], x2[n2], acc2[n2 * (n2 - 1) / 2 + m]);
          const float2 wp = make_float2(w[r][2 * i], w[r][2 * i + 1]);
#pragma unroll
          for (int m = 0; m < B; ++m) accp2[m] = __ffma2_rn(wp, x2[m], accp2[m]);
        }
      }
#pragma unroll
      for (int i = 0; i < BLK_PAIRS; ++i) acc[i] = acc2[i].x + acc2[i].y;
#pragma unroll
      for (int i = BLK_PAIRS; i < 32; ++i) acc[i] = 0.0f;
#pragma unroll
      for (int m = 0; m < B; ++m) accp[m] = accp2[m].x + accp2[m].y;
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
    const float pv_own = scratch[32 + n];  // margin of the sample this lane looks after
    __syncwarp();
    // ---- 8-step recurrence, every lane the same ----------------------------------------------------------
    float a_nv = tab[nv], dl = tab[32 + nv], apw_own = tab[n];
    if (DECAY) decaying_block_tables<B>((double)p.eta0, (double)p.lambda, first_j + b * B, nv, apw, cfac, apw_own, a_nv, dl);
    float t[B], beta[B], yv[B], cf[B], sc[B];
#pragma unroll
    for (int m = 0; m < B; ++m) yv[m] = __shfl_sync(0xffffffffu, y_cur, m);
    block8_constants<LOSS>(yv, apw, cfac, nv, sc, cf);
#pragma unroll
    for (int m = 0; m < B; ++m) {
      t[m] = sc[m] * pv[m];
#pragma unroll
      for (int k2 = 0; k2 < m; ++k2) Gs[m * (m - 1) / 2 + k2] *= sc[m];
    }
    // lane n & 7 expands the logistic factor of its own sample around t0_n (scratch[40..71] holds the expansions)
    block8_recurrence<LOSS>(t, Gs, cf, yv, y_cur * apw_own * 1.4426950408889634f * pv_own, (float4*)(scratch + 40), beta);
    // ---- w <- w - (1 - a^nv) w - sum_m gamma_m x_m,  gamma_m = beta_m a^nv ----------------------------------
    {
      constexpr int NP = XPairs<XT>::NP;
      float2 ngm2[B];
#pragma unroll
      for (int m = 0; m < B; ++m) {
        const float gm = -(beta[m] * a_nv);
        ngm2[m] = make_float2(gm, gm);
      }
      const float2 ndl2 = make_float2(-dl, -dl);
#pragma unroll
      for (int r = 0; r < R; ++r) {
#pragma unroll
        for (int i = 0; i < NP; ++i) {
          float2 wv = make_float2(w[r][2 * i], w[r][2 * i + 1]);
          wv = __ffma2_rn(ndl2, wv, wv);
#pragma unroll
          for (int m = 0; m < B; ++m) wv = __ffma2_rn(ngm2[m], XPairs<XT>::get(raw[r][m], i), wv);
          w[r][2 * i] = wv.x;
          w[r][2 * i + 1] = wv.y;
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
