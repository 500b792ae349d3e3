// Per-node SGD chains on dense rows, blocked form (see chain_block.cuh for the algebra), one CTA per node, with the
// Gram block of every block of samples computed by warps of its own.
//
// With few nodes a chain is bound by the dependent loop of a block: model update -> p = X_b w -> 8-step recurrence ->
// model update. The Gram block G_b = X_b X_b^T does not depend on the model; in chain_block_kernel the math warps
// form it while the recurrence runs, but it takes them about twice as long as the recurrence, so it ends up on the
// path. Here the math warps only keep the model (p and update), and "Gram warps" form the Gram block two blocks
// ahead, beside the math warps' part of the loop, so that the recurrence has the SM to itself: Gram warp c takes the
// 28 entries over the c-th group of 64 16-byte chunks (two chunks per lane). W math warps (32 chunks each) and ceil(chunks / 64) Gram warps: 14 warps for
// 256 chunks, which leaves every thread 128 registers (the recurrence warp needs about 120).
//
//                math warps                   Gram warps                           recurrence warp
//                w <- w - (1-a^B) w - ...     rows of block b+1: G_{b+1} partials   labels, constants of block b,
//                rows of block b -> regs      -> smem (buffer (b+1) & 1)           sum G_b partials (buffer b & 1)
//                p_b partials -> smem
//                ------------------------------ barrier 1 ---------------------------------------------------
//                -                            -                                    sum p_b, recurrence, gamma -> smem
//                ------------------------------ barrier 2 ---------------------------------------------------
// The copy warp (warp 1) requests rows with bulk asynchronous copies into a ring of stages (never multicast); the stage
// of block b is refilled after barrier 1 of block b, when the math warps hold its rows in registers and its Gram block is long done. Waits on arriving
// rows are bounded; a wait that runs out is flagged before a barrier and read by every warp right after barrier 2.
#pragma once

#include "chain_cluster.cuh"

namespace wpsgd {

constexpr int GRAM_MAX_MATH_WARPS = 8;
constexpr int GRAM_MAX_GROUPS = 4;  // groups of 64 chunks

struct GramSmem {
  size_t ring, redG, redP, totG, gam, tab, jet, bars, flag, total;
  __host__ __device__ GramSmem(int stages, size_t row_bytes) {
    ring = 0;
    redG = ring + (size_t)stages * BLK_B * row_bytes;                          // [2][groups][32]
    redP = redG + 2 * (size_t)GRAM_MAX_GROUPS * 32 * sizeof(float);            // [W][8]
    totG = redP + (size_t)GRAM_MAX_MATH_WARPS * BLK_B * sizeof(float);         // [32]
    gam = totG + 32 * sizeof(float);                                           // [16]
    tab = gam + 16 * sizeof(float);                                            // [48]
    jet = tab + 3 * 16 * sizeof(float);                                        // [8] float4
    bars = jet + 8 * 4 * sizeof(float);                                        // [8]
    flag = bars + 8 * sizeof(unsigned long long);
    total = flag + 16;
  }
};

// The 28 Gram entries (entry n(n-1)/2 + m, m < n) of 8 rows over one 16-byte chunk of columns, added to acc2.
template <typename XT>
__device__ __forceinline__ void gram_chunk(const uint4 (&raw)[BLK_B], float2 (&acc2)[BLK_PAIRS]) {
  constexpr int NP = XPairs<XT>::NP;
#pragma unroll
  for (int i = 0; i < NP; ++i) {
    float2 x2[BLK_B];
#pragma unroll
    for (int m = 0; m < BLK_B; ++m) x2[m] = XPairs<XT>::get(raw[m], i);
#pragma unroll
    for (int n2 = 1; n2 < BLK_B; ++n2)
#pragma unroll
      for (int m = 0; m < n2; ++m) acc2[n2 * (n2 - 1) / 2 + m] = __ffma2_rn(x2[m], x2[n2], acc2[n2 * (n2 - 1) / 2 + m]);
  }
}

template <typename XT, int LOSS>
__global__ void __launch_bounds__(64 + 32 * GRAM_MAX_MATH_WARPS + 32 * GRAM_MAX_GROUPS, 1) chain_gram_kernel(const BlockParams bp) {
  constexpr int V = XVec<XT>::V;
  constexpr int NP = XPairs<XT>::NP;
  constexpr int B = BLK_B;
  extern __shared__ __align__(16) unsigned char smem[];
  const ChainParams& p = bp.c;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int S = bp.stages;
  const int j = p.order[blockIdx.x];
  const long long n_run = p.n_steps[j];
  const long long d = p.d;
  const size_t row_bytes = (size_t)d * sizeof(XT);
  const size_t ld_bytes = (size_t)p.ld * sizeof(XT);
  const GramSmem L(S, row_bytes);
  unsigned char* ring = smem + L.ring;
  float* redG = (float*)(smem + L.redG);
  float* redP = (float*)(smem + L.redP);
  float* totG = (float*)(smem + L.totG);
  float* gam = (float*)(smem + L.gam);  // gamma_0..7, [8] = 1 - a^nv
  float* tab = (float*)(smem + L.tab);  // [0..8] a^k, [16..24] eta / a^{k+1}, [32..40] 1 - a^k
  float4* jets = (float4*)(smem + L.jet);
  unsigned long long* bars = (unsigned long long*)(smem + L.bars);
  volatile int* give_up = (volatile int*)(smem + L.flag);
  const char* shard = (const char*)p.X + (size_t)p.shard_off[j] * ld_bytes;
  const float* yshard = p.y + p.shard_off[j];
  const uint32_t* idx = p.idx + p.idx_off[j];
  const long long nb = (n_run + B - 1) / B;
  const int chunks = (int)(d / V);
  const int W = (chunks + 31) / 32;        // math warps
  const int GW = (chunks + 63) / 64;       // Gram warps
  // Which warp does what. Warp v of a CTA issues from scheduler v % 4. The recurrence (warp 0) is a dependent chain
  // that must not wait for issue slots, and the Gram warps are busy exactly while it runs, so the Gram warps take
  // warp numbers that are not multiples of 4; the math warps, idle during the recurrence, take the rest.
  int gram_index = -1, math_index = -1;
  if (warp >= 2) {
    const int zeros_before = (warp - 1) / 4;               // multiples of 4 in [2, warp)
    const int others_before = (warp - 2) - zeros_before;   // the other warp numbers in [2, warp)
    const int zeros_total = (2 + W + GW - 1) / 4;          // multiples of 4 in [2, 2 + W + GW)
    if ((warp & 3) != 0 && others_before < GW) gram_index = others_before;
    else math_index = (warp & 3) == 0 ? zeros_before : zeros_total + others_before - GW;
  }

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
  // partial-sum slots that no warp writes stay zero
  for (int i = threadIdx.x; i < 2 * GRAM_MAX_GROUPS * 32; i += blockDim.x) redG[i] = 0.0f;
  for (int i = threadIdx.x; i < GRAM_MAX_MATH_WARPS * B; i += blockDim.x) redP[i] = 0.0f;
  __syncthreads();  // tables and barriers are set up

  // wait (bounded) until the rows of a block have landed in their stage
  auto wait_rows = [&](int stg, uint32_t parity) __attribute__((always_inline)) {
    if (!mbar_wait_bounded(&bars[stg], parity, bp.spin_limit)) {
      set_status(p.status, DEV_TIMEOUT, 1, (long long)blockIdx.x);
      *give_up = 1;
    }
  };

  if (warp == 0) {
    // =========================== recurrence warp ========================================================
    // Every lane runs the whole recurrence on its own copy of the block's scalars (no shuffle inside the dependent
    // chain). Lane n & 7 looks after the label of sample n.
    const int n = lane & (B - 1);
    float y_nxt = 0.0f;
    uint32_t id_nxt = 0u;
    if (nb > 0) y_nxt = yshard[idx[n]];
    if (nb > 1) id_nxt = idx[B + n];
    float apw[B], cfac[B];
#pragma unroll
    for (int m = 0; m < B; ++m) { apw[m] = tab[m]; cfac[m] = tab[16 + m]; }
    __syncthreads();  // start-up barrier: G_0 partials are in place

    for (long long b = 0; b < nb; ++b) {
      const int nv = (int)((n_run - b * B) < (long long)B ? (n_run - b * B) : (long long)B);
      const float y_cur = y_nxt;
      if (b + 1 < nb) y_nxt = yshard[id_nxt];
      if (b + 2 < nb) id_nxt = idx[(b + 2) * B + n];
      const float a_nv = tab[nv], dl_nv = tab[32 + nv];
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
      // G_b: lane l adds entry l over the Gram warps (they finished it before barrier 1 of the previous block)
      float Gs[BLK_PAIRS];  // sc_n G_mn at [n(n-1)/2 + m], m < n
      {
        const float* rG = redG + (size_t)(b & 1) * GRAM_MAX_GROUPS * 32;
        float g = rG[lane];
#pragma unroll
        for (int w = 1; w < GRAM_MAX_GROUPS; ++w) g += rG[w * 32 + lane];
        totG[lane] = g;
        __syncwarp();
#pragma unroll
        for (int n2 = 1; n2 < B; ++n2)
#pragma unroll
          for (int m = 0; m < n2; ++m) {
            const int k = n2 * (n2 - 1) / 2 + m;
            Gs[k] = totG[k] * sc[n2];
          }
        __syncwarp();
      }
      __syncthreads();  // barrier 1: p_b partials are in place
      float psum = redP[n];
#pragma unroll
      for (int w = 1; w < GRAM_MAX_MATH_WARPS; ++w) psum += redP[w * B + n];
      float t[B], beta[B];
#pragma unroll
      for (int m = 0; m < B; ++m) t[m] = sc[m] * __shfl_sync(0xffffffffu, psum, m);
      if (LOSS == LOSS_LOGISTIC) {
        // lane n & 7 expands the factor of its own sample around t0_n; every lane then fetches all eight expansions
        if (lane < B) jets[lane] = logistic_jet(y_cur * tab[n] * 1.4426950408889634f * psum);
        __syncwarp();
        float4 jet[B];
        float dlt[B];
#pragma unroll
        for (int m = 0; m < B; ++m) {
          jet[m] = jets[m];
          dlt[m] = 0.0f;
        }
        float dmax = 0.0f;
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
            for (int k = 0; k < B; ++k)
              if (k == m) { tm_ = t[k]; cfm = cf[k]; }
            const float bm = cfm * logistic_factor(tm_);
#pragma unroll
            for (int k = 0; k < B; ++k)
              if (k == m) beta[k] = bm;
#pragma unroll
            for (int n2 = 1; n2 < B; ++n2)
#pragma unroll
              for (int k = 0; k < n2; ++k)
                if (k == m) t[n2] = fmaf(-bm, Gs[n2 * (n2 - 1) / 2 + k], t[n2]);
          }
        }
      } else {
#pragma unroll
        for (int m = 0; m < B; ++m) {
          if (LOSS == LOSS_HINGE) {
            beta[m] = (t[m] < 1.0f) ? cf[m] : 0.0f;
          } else {
            beta[m] = cf[m] * (t[m] - yv[m]);
          }
#pragma unroll
          for (int n2 = m + 1; n2 < B; ++n2) t[n2] = fmaf(-beta[m], Gs[n2 * (n2 - 1) / 2 + m], t[n2]);
        }
      }
      // gamma_m = eta g_m a^{nv-1-m} = beta_m a^{nv}
      float mine = dl_nv;
#pragma unroll
      for (int m = 0; m < B; ++m)
        if (lane == m) mine = beta[m] * a_nv;
      if (lane <= B) gam[lane] = mine;
      __syncthreads();  // barrier 2: gamma published, G_{b+1} partials in place
      if (*give_up) break;
    }
    return;
  }

  if (warp == 1) {
    // =========================== copy warp ==============================================================
    // Lane m < 8 requests row m of a block as one bulk copy; the eight copies complete on the stage's barrier.
    const uint32_t copy_bytes = (uint32_t)row_bytes;
    uint32_t id_next = 0u;
    auto peek = [&](long long blk) __attribute__((always_inline)) {
      if (lane < B && blk < nb) id_next = idx[blk * B + lane];
    };
    auto request = [&](long long blk, int stg) __attribute__((always_inline)) {
      if (blk < nb && blk != bp.drop_block) {
        if (lane == 0) mbar_arrive_expect_tx(&bars[stg], B * copy_bytes);
        __syncwarp();
        if (lane < B)
          bulk_copy_g2s(ring + ((size_t)stg * B + lane) * row_bytes, shard + (size_t)id_next * ld_bytes, copy_bytes, &bars[stg]);
      }
    };
    long long requested = 0;
    for (int s = 0; s < S; ++s) {
      peek(s);
      request(s, s);
      ++requested;
    }
    peek(requested);
    __syncthreads();  // start-up barrier: the math warps hold block 0 in registers, its Gram block is done
    int st = 0;       // stage of block b
    long long b = 0;
    bool stop = false;
    for (; b < nb; ++b) {
      if (b >= 1) __syncthreads();  // barrier 1 of block b (block 0: the start-up barrier stands in for it)
      // the rows of block b are in the math warps' registers and its Gram block is done: its stage takes block b + S
      request(requested, st);
      ++requested;
      peek(requested);
      st = (st + 1 == S) ? 0 : st + 1;
      if (b == 0) __syncthreads();  // barrier 1 of block 0
      __syncthreads();              // barrier 2
      if (*give_up) { stop = true; break; }
    }
    if (stop) {
      // leave no copy in flight into this CTA's shared memory: wait (bounded) on the stage of every block that was
      // requested and may not have landed yet
      for (long long blk = b; blk < requested && blk < nb; ++blk)
        if (blk != bp.drop_block) mbar_wait_bounded(&bars[blk % S], (uint32_t)((blk / S) & 1), bp.spin_limit);
    }
    return;
  }

  if (gram_index >= 0) {
    // =========================== Gram warps ==============================================================
    const int gw = gram_index;
    const int grp = gw;
    // Gram block of block g (its rows awaited, bounded) -> buffer g & 1
    auto gram_of = [&](long long g) __attribute__((always_inline)) {
      wait_rows((int)(g % S), (uint32_t)((g / S) & 1));
      const unsigned char* stage = ring + (size_t)(g % S) * B * row_bytes;
      float* out = redG + ((size_t)(g & 1) * GRAM_MAX_GROUPS + grp) * 32;
      float2 acc2[BLK_PAIRS];
#pragma unroll
      for (int k = 0; k < BLK_PAIRS; ++k) acc2[k] = make_float2(0.0f, 0.0f);
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        const int chunk = grp * 64 + r * 32 + lane;
        if (chunk < chunks) {
          uint4 raw[B];
#pragma unroll
          for (int m = 0; m < B; ++m) raw[m] = *(const uint4*)(stage + (size_t)m * row_bytes + (size_t)chunk * 16);
          gram_chunk<XT>(raw, acc2);
        }
      }
      float part[32];
#pragma unroll
      for (int k = 0; k < BLK_PAIRS; ++k) part[k] = acc2[k].x + acc2[k].y;
#pragma unroll
      for (int k = BLK_PAIRS; k < 32; ++k) part[k] = 0.0f;
      out[lane] = warp_transpose_sum32(part);  // lane l: entry l over the warp's columns
    };
    if (nb > 0) gram_of(0);
    if (nb > 1) gram_of(1);
    __syncthreads();  // start-up barrier
    for (long long b = 0; b < nb; ++b) {
      __syncthreads();  // barrier 1: the recurrence warp has read the Gram block of block b (buffer b & 1)
      __syncthreads();  // barrier 2
      if (*give_up) break;
      if (b + 2 < nb) gram_of(b + 2);  // beside the math warps' update and p, done before barrier 1 of block b + 1
    }
    return;
  }

  // ============================= math warps ==============================================================
  const int mw = math_index;
  const long long c0 = ((long long)mw * 32 + lane) * V;
  const bool act = c0 < d;
  float2 w2[NP];
#pragma unroll
  for (int i = 0; i < NP; ++i) w2[i] = make_float2(0.0f, 0.0f);
  if (act) {
    const float* src = p.resume ? (p.W + (size_t)j * d + c0) : (p.w0 ? p.w0 + c0 : nullptr);
    if (src) {
#pragma unroll
      for (int i = 0; i < NP; ++i) w2[i] = make_float2(src[2 * i], src[2 * i + 1]);
    }
  }
  uint4 cur[B];
  auto load_rows = [&](int stg) __attribute__((always_inline)) {
    const unsigned char* stage = ring + (size_t)stg * B * row_bytes;
#pragma unroll
    for (int m = 0; m < B; ++m)
      cur[m] = act ? *(const uint4*)(stage + (size_t)m * row_bytes + (size_t)(mw * 32 + lane) * 16) : make_uint4(0u, 0u, 0u, 0u);
  };
#pragma unroll
  for (int m = 0; m < B; ++m) cur[m] = make_uint4(0u, 0u, 0u, 0u);
  if (nb > 0) {
    wait_rows(0, 0u);
    load_rows(0);
  }
  __syncthreads();  // start-up barrier
  int st = (S > 1) ? 1 : 0;          // stage of block b + 1 ...
  uint32_t par = (S > 1) ? 0u : 1u;  // ... and the parity of the barrier phase that brings it
  for (long long b = 0; b < nb; ++b) {
    // ---- p_b = X_b w over this thread's columns ---------------------------------------------------------------
    float2 a2[B];
#pragma unroll
    for (int m = 0; m < B; ++m) a2[m] = make_float2(0.0f, 0.0f);
#pragma unroll
    for (int i = 0; i < NP; ++i)
#pragma unroll
      for (int m = 0; m < B; ++m) a2[m] = __ffma2_rn(w2[i], XPairs<XT>::get(cur[m], i), a2[m]);
    float accp[B];
#pragma unroll
    for (int m = 0; m < B; ++m) accp[m] = a2[m].x + a2[m].y;
    const float ptot = warp_transpose_sum8(accp);  // every lane: p_{lane >> 2} over the warp's columns
    if ((lane & 3) == 0) redP[mw * B + (lane >> 2)] = ptot;
    __syncthreads();  // barrier 1
    __syncthreads();  // barrier 2: gamma_b is in gam
    if (*give_up) break;
    // ---- w <- w - (1 - a^nv) w - sum_m gamma_m x_m ---------------------------------------------------------------
    {
      float2 ngm2[B];
#pragma unroll
      for (int m = 0; m < B; ++m) {
        const float g = -gam[m];
        ngm2[m] = make_float2(g, g);
      }
      const float ndl = -gam[B];
      const float2 ndl2 = make_float2(ndl, ndl);
#pragma unroll
      for (int i = 0; i < NP; ++i) {
        float2 wv = __ffma2_rn(ndl2, w2[i], w2[i]);
#pragma unroll
        for (int m = 0; m < B; ++m) wv = __ffma2_rn(ngm2[m], XPairs<XT>::get(cur[m], i), wv);
        w2[i] = wv;
      }
    }
    // ---- rows of block b + 1 (the Gram warps have waited for them already) -> registers --------------------------------
    if (b + 1 < nb) {
      wait_rows(st, par);
      load_rows(st);
    }
    if (++st == S) { st = 0; par ^= 1u; }
  }

  if (act) {
    float* dst = p.W + (size_t)j * d + c0;
#pragma unroll
    for (int i = 0; i < NP; ++i) {
      dst[2 * i] = w2[i].x;
      dst[2 * i + 1] = w2[i].y;
    }
  }
}

}  // namespace wpsgd
