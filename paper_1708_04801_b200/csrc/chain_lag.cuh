// Per-node SGD chains on dense bf16 rows, blocked form with the margins taken one block behind the model
// ("lagged" form), columns of a chain split over the CTAs of a thread-block cluster.
//
// In the blocked form (chain_block.cuh) a block of B = 8 samples x_0..x_7 with model w at its start needs
// p_n = w.x_n and G_mn = x_m.x_n before its scalar recurrence, and the model after it is a^B w - sum_m gamma_m x_m.
// p depends on the model, so model update -> p -> exchange -> recurrence -> model update is one dependent loop per
// block, and a chain is as slow as that loop. Substituting the update of the previous block into p,
//     p_n = a^B (w_prev . x_n) - sum_m gamma_prev_m (x_prev_m . x_n) = a^B q_n - sum_m gamma_prev_m C_mn,
// with w_prev the model at the start of the previous block, q_n = w_prev . x_n and C the 8 x 8 products between the
// rows of the previous block and this one. These are the iterates of Eq. 5 exactly (in exact arithmetic). q_n needs
// the model only as it was one block earlier, and C and G need no model at all. The dependent loop now spans two
// blocks (gamma_{b-1} -> w_b -> q_{b+1} -> gamma_{b+1}) while the recurrences themselves follow one another directly.
//
// Work split (per CTA; CTA `rank` of a cluster of C owns the 16-byte chunks [rank cpc, (rank + 1) cpc) of every row):
//   warp 0      recurrence warp: waits for the partial sums of block b (q_b; G_b and C_{b-1,b}), adds them over all
//               math warps of the cluster, p = a^B q - C^T gamma_{b-1}, 8-step recurrence, publishes gamma_b
//   warp 1      copy warp: bulk asynchronous copies of the CTA's column slice of the 8 rows of a block into a ring of
//               stages (a "landed" barrier and a "free" barrier per stage; never multicast)
//   math warps  iteration i:  [G_{i+1} ; C_{i,i+1}] = [X_{i+1} ; X_i] X_{i+1}^T over the warp's 256 columns on the
//               tensor cores (bf16 products are exact, fp32 accumulation; one m16n8k16 per 16 columns);
//               wait for gamma_i;  w <- a^nv w - sum_m gamma_m x_m (rows of block i held in registers);
//               q_{i+2} = w . X_{i+2} over the thread's columns (packed fp32 FMAs), summed over the warp.
//               Partial sums go to the tables of EVERY CTA of the cluster with st.async, which reports the bytes to
//               a barrier of the destination CTA; every CTA runs the recurrence redundantly, so nothing comes back.
// Flow control. The partial-sum tables and their barriers are four deep (block number mod 4). A math warp sends the
// G / C sums of block i + 1 after it has seen gamma_{i-1} of its own CTA, which needed the q_{i-1} of every CTA, which
// those sent after seeing their own gamma_{i-3}: the recurrence warp of any CTA of the cluster is then at block i - 2
// or later, so the blocks whose sums it has not read yet are among i - 2 .. i + 1, four different tables. The same
// count holds for q (sent for block i + 2 after gamma_i; every recurrence warp is at block i - 1 or later). gamma
// itself stays inside its CTA and is double buffered: gamma_{i+2} needs q_{i+2}, which is formed after gamma_i was read.
//
// gamma_b goes from the recurrence warp to the math warps of its CTA through a named hardware barrier (the math
// warps park there without polling; the recurrence warp only arrives). Every wait on data from elsewhere (rows,
// partial sums, free stages) is a bounded poll that also ends when the give-up flag is set. A wait that
// runs out sets the status word and the flag of every CTA of the cluster; math warps carry on with whatever is in
// shared memory until the recurrence warp, which samples the flag once per block, publishes "stop" with gamma: it
// never leaves without arriving at the barrier, so nobody is left parked. All threads meet at one final cluster
// barrier, so no CTA exits while a peer may still store into its shared memory.
#pragma once

#include "chain_mma.cuh"

namespace wpsgd {

constexpr int LAG_SLOTS = 16;     // math warps of a whole cluster
constexpr int LAG_DEPTH = 4;      // partial-sum tables in flight (block number mod 4)
constexpr int LAG_GC_VALS = 128;  // accumulator rows 0..7 (G) then rows 8..15 (products with the previous block)
constexpr uint32_t LAG_GC_BYTES = LAG_GC_VALS * sizeof(float);  // one math warp -> one CTA, per block
constexpr uint32_t LAG_Q_BYTES = BLK_B * sizeof(float);

struct LagSmem {
  size_t row_stride, ring, redGC, redQ, tot, gam, tab, jet, full, fre, gbar, qbar, flag, total;
  __host__ __device__ LagSmem(int stages, size_t slice_bytes) {
    row_stride = slice_bytes + 16;
    ring = 0;
    redGC = ring + (size_t)stages * BLK_B * row_stride;                   // [4][slots][128]
    redQ = redGC + LAG_DEPTH * (size_t)LAG_SLOTS * LAG_GC_VALS * sizeof(float);   // [4][slots][8]
    tot = redQ + LAG_DEPTH * (size_t)LAG_SLOTS * BLK_B * sizeof(float);   // [128]
    gam = tot + LAG_GC_VALS * sizeof(float);                              // [2][16]: gamma_0..7, 1 - a^nv, stop
    tab = gam + 2 * 16 * sizeof(float);                                   // [48]
    jet = tab + 3 * 16 * sizeof(float);                                   // [8] float4
    full = jet + 8 * 4 * sizeof(float);                                   // [8] rows of a stage have landed
    fre = full + 8 * sizeof(unsigned long long);                          // [8] stage may be refilled
    gbar = fre + 8 * sizeof(unsigned long long);                          // [4] G / C partial sums
    qbar = gbar + LAG_DEPTH * sizeof(unsigned long long);                 // [4] q partial sums
    flag = qbar + LAG_DEPTH * sizeof(unsigned long long);
    total = flag + 16;
  }
};

// Named hardware barrier `id` of the CTA for `nthreads` threads: sync parks the warp until all have arrived, arrive
// only reports. Stores before an arrive are visible after the matching sync.
__device__ __forceinline__ void named_bar_sync(int id, int nthreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}
__device__ __forceinline__ void named_bar_arrive(int id, int nthreads) {
  asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
  const uint32_t a = (uint32_t)__cvta_generic_to_shared(bar);
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(a) : "memory");
}
__device__ __forceinline__ void st_async_f32(uint32_t addr, float a, uint32_t mbar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.f32 [%0], %1, [%2];" ::"r"(addr), "f"(a),
               "r"(mbar)
               : "memory");
}
// Non-blocking look at a barrier phase (try_wait may hold the thread for a while even when the phase is complete).
__device__ __forceinline__ bool mbar_test_wait(unsigned long long* bar, uint32_t parity, bool cluster_scope) {
  const uint32_t a = (uint32_t)__cvta_generic_to_shared(bar);
  uint32_t ok;
  if (cluster_scope)
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(a), "r"(parity)
        : "memory");
  else
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(a), "r"(parity)
        : "memory");
  return ok != 0;
}
// Bounded wait that also ends when the give-up flag is set; true when the phase completed.
__device__ __forceinline__ bool mbar_wait_or_give_up(unsigned long long* bar, uint32_t parity, long long limit,
                                                     volatile int* give_up, bool cluster_scope) {
  for (long long i = 0; i < limit; ++i) {
    if (mbar_test_wait(bar, parity, cluster_scope)) return true;
    if (*give_up) return false;
  }
  return false;
}

template <int LOSS>
__global__ void __launch_bounds__(64 + 32 * 8, 1) chain_lag_kernel(const ClusterParams cp) {
  constexpr int B = BLK_B;
  extern __shared__ __align__(16) unsigned char smem[];
  const BlockParams& bp = cp.b;
  const ChainParams& p = bp.c;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int math_warps = (blockDim.x >> 5) - 2;
  const int S = bp.stages;
  const uint32_t C = cluster_nctarank(), rank = cluster_ctarank();
  const int j = p.order[blockIdx.x / C];
  const long long n_run = p.n_steps[j];
  const long long d = p.d;
  const long long chunks = d / 8;
  const long long chunk0 = (long long)rank * cp.chunks_per_cta;
  const long long chunk_end = chunk0 + cp.chunks_per_cta < chunks ? chunk0 + cp.chunks_per_cta : chunks;
  const int my_chunks = (int)(chunk_end > chunk0 ? chunk_end - chunk0 : 0);
  const size_t slice_bytes = (size_t)cp.chunks_per_cta * 16;
  const size_t ld_bytes = (size_t)p.ld * 2;
  const LagSmem L(S, slice_bytes);
  const size_t row_stride = L.row_stride;
  unsigned char* ring = smem + L.ring;
  float* redGC = (float*)(smem + L.redGC);
  float* redQ = (float*)(smem + L.redQ);
  float* tot = (float*)(smem + L.tot);
  float* gam = (float*)(smem + L.gam);
  float* tab = (float*)(smem + L.tab);  // [0..8] a^k, [16..24] eta / a^{k+1}, [32..40] 1 - a^k
  float4* jets = (float4*)(smem + L.jet);
  unsigned long long* full = (unsigned long long*)(smem + L.full);
  unsigned long long* fre = (unsigned long long*)(smem + L.fre);
  unsigned long long* gbar = (unsigned long long*)(smem + L.gbar);
  unsigned long long* qbar = (unsigned long long*)(smem + L.qbar);
  volatile int* give_up = (volatile int*)(smem + L.flag);
  const char* shard = (const char*)p.X + (size_t)p.shard_off[j] * ld_bytes + (size_t)chunk0 * 16;
  const float* yshard = p.y + p.shard_off[j];
  const uint32_t* idx = p.idx + p.idx_off[j];
  const long long nb = (n_run + B - 1) / B;

  // ---- set-up --------------------------------------------------------------------------------------------------
  if (threadIdx.x <= B) {  // power tables in fp64, rounded once
    const double a = 1.0 - bp.eta_lambda;
    double pw = 1.0;
    for (int k = 0; k < (int)threadIdx.x; ++k) pw *= a;
    tab[threadIdx.x] = (float)pw;
    tab[16 + threadIdx.x] = (float)((double)p.eta0 / (pw * a));
    tab[32 + threadIdx.x] = (float)(1.0 - pw);
  }
  if (threadIdx.x == 32) {
    for (int s = 0; s < S; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&fre[s], math_warps);
    }
    for (int q = 0; q < LAG_DEPTH; ++q) {
      mbar_init(&gbar[q], 1);
      mbar_init(&qbar[q], 1);
    }
    *give_up = 0;
    mbar_fence_init();
  }
  {
    // ring and partial-sum tables start at zero: columns beyond a slice and the table slots that no math warp
    // writes are never written later
    uint4* z = (uint4*)smem;
    const int n16 = (int)(L.tot / 16);
    for (int i = threadIdx.x; i < n16; i += blockDim.x) z[i] = make_uint4(0u, 0u, 0u, 0u);
  }
  fence_proxy_async_shared();
  __syncthreads();

  const int gamma_threads = 32 * (math_warps + 1);  // recurrence warp and math warps meet at the gamma barriers 1 and 2
  auto flag_timeout = [&](int where) __attribute__((always_inline)) {
    set_status(p.status, DEV_TIMEOUT, where, (long long)blockIdx.x);
    for (uint32_t rr = 0; rr < C; ++rr) st_shared_cluster(map_shared_rank((const void*)give_up, rr), 1);
  };

  if (warp == 0) {
    // =========================== recurrence warp ========================================================
    const int n = lane & (B - 1);
    float y_nxt = 0.0f;
    uint32_t id_nxt = 0u;
    if (nb > 0) y_nxt = yshard[idx[n]];
    if (nb > 1) id_nxt = idx[B + n];
    float apw[B], cfac[B], gprev[B];
#pragma unroll
    for (int m = 0; m < B; ++m) { apw[m] = tab[m]; cfac[m] = tab[16 + m]; gprev[m] = 0.0f; }
    const float a_full = tab[B];
    const uint32_t slots = C * (uint32_t)math_warps;
    cluster_barrier();  // start-up: every CTA of the cluster runs and has set up its shared memory

    for (long long b = 0; b < nb; ++b) {
      const int nv = (int)((n_run - b * B) < (long long)B ? (n_run - b * B) : (long long)B);
      const int q = (int)(b & (LAG_DEPTH - 1));
      const uint32_t parity = (uint32_t)((b / LAG_DEPTH) & 1);
      if (lane == 0) {
        mbar_arrive_expect_tx(&gbar[q], slots * LAG_GC_BYTES);
        mbar_arrive_expect_tx(&qbar[q], slots * LAG_Q_BYTES);
      }
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
      // ---- G_b and C_{b-1,b}: sum over the math warps of the cluster ---------------------------------------------
      bool stop = false;
      if (!mbar_wait_or_give_up(&gbar[q], parity, bp.spin_limit, give_up, true)) {
        if (!*give_up) flag_timeout(2);
        stop = true;
      }
      float Gs[BLK_PAIRS];  // sc_n G_mn at [n(n-1)/2 + m], m < n
      float pcorr = 0.0f;   // lane n: sum_m gamma_prev_m C_mn
      {
        const float4* rGC = (const float4*)(redGC + (size_t)q * LAG_SLOTS * LAG_GC_VALS) + lane;
        float4 s4 = rGC[0];
#pragma unroll
        for (int w = 1; w < LAG_SLOTS; ++w) {
          const float4 v = rGC[w * (LAG_GC_VALS / 4)];
          s4.x += v.x; s4.y += v.y; s4.z += v.z; s4.w += v.w;
        }
        ((float4*)tot)[lane] = s4;
        __syncwarp();
#pragma unroll
        for (int n2 = 1; n2 < B; ++n2) {
          const float4 lo = *(const float4*)&tot[n2 * 8], hi = *(const float4*)&tot[n2 * 8 + 4];
          const float row[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
#pragma unroll
          for (int m = 0; m < n2; ++m) Gs[n2 * (n2 - 1) / 2 + m] = row[m] * sc[n2];
        }
#pragma unroll
        for (int m = 0; m < B; ++m) pcorr = fmaf(gprev[m], tot[64 + m * 8 + n], pcorr);
        __syncwarp();
      }
      // ---- q_b, then p_b = a^B q_b - C^T gamma_{b-1} (b = 0: p = q) -----------------------------------------------
      if (!stop && !mbar_wait_or_give_up(&qbar[q], parity, bp.spin_limit, give_up, true)) {
        if (!*give_up) flag_timeout(3);
        stop = true;
      }
      if (*give_up) stop = true;
      float psum;
      {
        const float* rQ = redQ + (size_t)q * LAG_SLOTS * B + n;
        float qs = rQ[0];
#pragma unroll
        for (int w = 1; w < LAG_SLOTS; ++w) qs += rQ[w * B];
        psum = (b == 0) ? qs : fmaf(a_full, qs, -pcorr);  // lane l: p of sample l & 7
      }
      float t[B], beta[B];
#pragma unroll
      for (int m = 0; m < B; ++m) t[m] = sc[m] * __shfl_sync(0xffffffffu, psum, m);
      if (LOSS == LOSS_LOGISTIC) {
        // lane n < 8 expands the factor of its own sample around t0_n; every lane then fetches all eight expansions
        if (lane < B) jets[lane] = logistic_jet(y_cur * tab[n] * 1.4426950408889634f * psum);
        __syncwarp();
        float4 jet[B];
        float dlt[B];
#pragma unroll
        for (int m = 0; m < B; ++m) {
          jet[m] = jets[m];
          dlt[m] = 0.0f;
        }
        __syncwarp();
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
      // gamma_m = eta g_m a^{nv-1-m} = beta_m a^{nv}; [8] = 1 - a^nv; [9] = leave after this block
      float mine = dl_nv;
#pragma unroll
      for (int m = 0; m < B; ++m) {
        gprev[m] = beta[m] * a_nv;
        if (lane == m) mine = gprev[m];
      }
      if (lane == B + 1) mine = stop ? 1.0f : 0.0f;
      if (lane <= B + 1) gam[(b & 1) * 16 + lane] = mine;
      if (b & 1) named_bar_arrive(2, gamma_threads);  // gamma_b published
      else named_bar_arrive(1, gamma_threads);
      if (stop) break;
    }
    cluster_barrier();  // nobody exits while a peer may still store into its shared memory
    return;
  }

  if (warp == 1) {
    // =========================== copy warp ==============================================================
    // Lane m < 8 requests this CTA's column slice of row m of a block as one bulk copy; the eight copies complete on
    // the stage's "landed" barrier. A stage is refilled once every math warp has reported that it is done with it.
    const uint32_t copy_bytes = (uint32_t)my_chunks * 16u;
    uint32_t id_next = 0u;
    auto peek = [&](long long blk) __attribute__((always_inline)) {
      if (lane < B && blk < nb) id_next = idx[blk * B + lane];
    };
    auto request = [&](long long blk, int stg) __attribute__((always_inline)) {
      if (blk < nb && blk != bp.drop_block && copy_bytes > 0) {
        if (lane == 0) mbar_arrive_expect_tx(&full[stg], B * copy_bytes);
        __syncwarp();
        if (lane < B)
          bulk_copy_g2s(ring + ((size_t)stg * B + lane) * row_stride, shard + (size_t)id_next * ld_bytes, copy_bytes, &full[stg]);
      }
    };
    long long requested = 0;
    for (int s = 0; s < S; ++s) {
      peek(s);
      request(s, s);
      ++requested;
    }
    peek(requested);
    cluster_barrier();  // start-up
    int st = 0;         // stage of block i
    bool gave_up = false;
    for (long long i = 0; requested < nb; ++i) {
      // block i has been used up by the math warps: its stage takes block i + S
      if (!mbar_wait_or_give_up(&fre[st], (uint32_t)((i / S) & 1), bp.spin_limit, give_up, false)) {
        if (!*give_up) flag_timeout(4);
        gave_up = true;
        break;
      }
      request(requested, st);
      ++requested;
      peek(requested);
      st = (st + 1 == S) ? 0 : st + 1;
    }
    if (gave_up || *give_up) {
      // leave no copy in flight into this CTA's shared memory: wait (bounded) on every stage; a stage whose latest
      // request has landed answers at once
      if (copy_bytes > 0)
        for (long long blk = requested > S ? requested - S : 0; blk < requested && blk < nb; ++blk)
          if (blk != bp.drop_block) mbar_wait_bounded(&full[blk % S], (uint32_t)((blk / S) & 1), bp.spin_limit);
    }
    cluster_barrier();
    return;
  }

  // ============================= math warps ==============================================================
  const int mw = warp - 2;
  const int lc = mw * 32 + lane;  // this thread's chunk within the CTA's slice
  const bool act = lc < my_chunks;
  const int warp_chunks = my_chunks - mw * 32 < 0 ? 0 : (my_chunks - mw * 32 > 32 ? 32 : my_chunks - mw * 32);
  const int ksteps = (warp_chunks + 1) >> 1;  // 16 columns (two chunks) per tensor-core instruction
  float2 w2[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) w2[i] = make_float2(0.0f, 0.0f);
  if (act) {
    const long long c0 = (chunk0 + lc) * 8;
    const float* src = p.resume ? (p.W + (size_t)j * d + c0) : (p.w0 ? p.w0 + c0 : nullptr);
    if (src) {
#pragma unroll
      for (int i = 0; i < 4; ++i) w2[i] = make_float2(src[2 * i], src[2 * i + 1]);
    }
  }
  // tile addresses of the tensor-core operand loads: lanes 8t..8t+7 give the 8 row addresses of tile t; tiles 0 and 2
  // are the rows of the newer block (columns +0 and +8), tiles 1 and 3 those of the older block
  const int tile = lane >> 3, trow = lane & 7;
  const size_t tile_off = (size_t)trow * row_stride + (size_t)mw * 512 + (size_t)(tile >> 1) * 16;
  const int slot = (int)rank * math_warps + mw;
  const uint32_t own_base = (uint32_t)__cvta_generic_to_shared(smem);
  bool alive = true;  // false once the recurrence warp has published "stop"

  auto wait_rows = [&](long long blk) __attribute__((always_inline)) {
    if (my_chunks > 0 && !mbar_wait_or_give_up(&full[blk % S], (uint32_t)((blk / S) & 1), bp.spin_limit, give_up, false)) {
      if (!*give_up) flag_timeout(1);
    }
  };
  // [G_new ; C_old,new] over this warp's columns -> table of block blk_new in every CTA of the cluster
  auto gram_pass = [&](long long blk_new, long long blk_old) __attribute__((always_inline)) {
    const unsigned char* src = ring + (size_t)(((tile & 1) ? blk_old : blk_new) % S) * B * row_stride + tile_off;
    // eight independent accumulators, two rounds of eight
    // 16-column steps; the operand tiles are loaded four at a time
    float acc[8][4];
#pragma unroll
    for (int a = 0; a < 8; ++a)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[a][e] = 0.0f;
#pragma unroll
    for (int round = 0; round < 4; ++round) {
      uint32_t q[4][4];
#pragma unroll
      for (int a = 0; a < 4; ++a)
        if (round * 4 + a < ksteps) ldmatrix_x4(q[a], src + (size_t)(round * 4 + a) * 32);
#pragma unroll
      for (int a = 0; a < 4; ++a)
        if (round * 4 + a < ksteps)
          mma_bf16_m16n8k16(acc[(round & 1) * 4 + a], q[a][0], q[a][1], q[a][2], q[a][3], q[a][0], q[a][2]);
    }
#pragma unroll
    for (int h = 4; h >= 1; h >>= 1)
#pragma unroll
      for (int a = 0; a < h; ++a)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[a][e] += acc[a + h][e];
    // accumulator rows 0..7: lane l holds G[l / 4][2 (l % 4) .. +1]; rows 8..15: C[l / 4][2 (l % 4) .. +1]
    const int q = (int)(blk_new & (LAG_DEPTH - 1));
    const uint32_t og = (uint32_t)__cvta_generic_to_shared(redGC + ((size_t)q * LAG_SLOTS + slot) * LAG_GC_VALS + lane * 2) - own_base;
    const uint32_t ob = (uint32_t)__cvta_generic_to_shared(&gbar[q]) - own_base;
    for (uint32_t rr = 0; rr < C; ++rr) {
      const uint32_t peer = map_shared_rank(smem, rr);  // the same offsets apply inside every CTA's window
      st_async_f32x2(peer + og, acc[0][0], acc[0][1], peer + ob);
      st_async_f32x2(peer + og + 64 * (uint32_t)sizeof(float), acc[0][2], acc[0][3], peer + ob);
    }
  };
  // this thread's columns of the rows of block blk into registers; q = w . x over them, summed over the warp,
  // -> table of block blk in every CTA of the cluster
  auto q_pass = [&](long long blk, uint4 (&raw)[B]) __attribute__((always_inline)) {
    const unsigned char* stage = ring + (size_t)(blk % S) * B * row_stride;
#pragma unroll
    for (int m = 0; m < B; ++m)
      raw[m] = act ? *(const uint4*)(stage + (size_t)m * row_stride + (size_t)lc * 16) : make_uint4(0u, 0u, 0u, 0u);
    float2 a2[B];
#pragma unroll
    for (int m = 0; m < B; ++m) a2[m] = make_float2(0.0f, 0.0f);
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int m = 0; m < B; ++m) a2[m] = __ffma2_rn(w2[i], XPairs<__nv_bfloat16>::get(raw[m], i), a2[m]);
    float accp[B];
#pragma unroll
    for (int m = 0; m < B; ++m) accp[m] = a2[m].x + a2[m].y;
    const float qtot = warp_transpose_sum8(accp);  // every lane: q_{lane >> 2} over the warp's columns
    const int q = (int)(blk & (LAG_DEPTH - 1));
    const uint32_t oq = (uint32_t)__cvta_generic_to_shared(redQ + ((size_t)q * LAG_SLOTS + slot) * B + (lane >> 2)) - own_base;
    const uint32_t ob = (uint32_t)__cvta_generic_to_shared(&qbar[q]) - own_base;
    if ((lane & 3) == 0) {
      for (uint32_t rr = 0; rr < C; ++rr) {
        const uint32_t peer = map_shared_rank(smem, rr);
        st_async_f32(peer + oq, qtot, peer + ob);
      }
    }
  };
  // w <- w - (1 - a^nv) w - sum_m gamma_m x_m with the rows of block i held in raw
  auto update = [&](long long i, const uint4 (&raw)[B]) __attribute__((always_inline)) {
    const float* g = gam + (i & 1) * 16;
    float2 ngm2[B];
#pragma unroll
    for (int m = 0; m < B; ++m) {
      const float v = -g[m];
      ngm2[m] = make_float2(v, v);
    }
    const float ndl = -g[B];
    const float2 ndl2 = make_float2(ndl, ndl);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      float2 wv = __ffma2_rn(ndl2, w2[k], w2[k]);
#pragma unroll
      for (int m = 0; m < B; ++m) wv = __ffma2_rn(ngm2[m], XPairs<__nv_bfloat16>::get(raw[m], k), wv);
      w2[k] = wv;
    }
  };
  // iteration i; raw holds the rows of block i on entry and those of block i + 2 on exit
  auto iteration = [&](long long i, uint4 (&raw)[B]) __attribute__((always_inline)) {
    if (i + 1 < nb) {
      wait_rows(i + 1);
      gram_pass(i + 1, i);
    }
    // nothing in shared memory of block i is read after this point
    __syncwarp();
    if (lane == 0) mbar_arrive(&fre[i % S]);
    if (i & 1) named_bar_sync(2, gamma_threads);  // gamma_i and the decision are in gam
    else named_bar_sync(1, gamma_threads);
    if (gam[(i & 1) * 16 + B + 1] != 0.0f) {
      alive = false;
      return;
    }
    update(i, raw);
    if (i + 2 < nb) {
      wait_rows(i + 2);
      q_pass(i + 2, raw);
    }
  };

  cluster_barrier();  // start-up

  uint4 raw_even[B], raw_odd[B];
#pragma unroll
  for (int m = 0; m < B; ++m) raw_even[m] = raw_odd[m] = make_uint4(0u, 0u, 0u, 0u);
  if (nb > 0) {
    wait_rows(0);
    q_pass(0, raw_even);  // p of block 0
    gram_pass(0, 0);      // G of block 0 (the other half of the table is not used for block 0)
  }
  if (nb > 1) {
    wait_rows(1);
    q_pass(1, raw_odd);  // q of block 1 against the starting model
  }
  for (long long i = 0; i < nb && alive; i += 2) {
    iteration(i, raw_even);
    if (i + 1 < nb && alive) iteration(i + 1, raw_odd);
  }
  cluster_barrier();

  if (act) {
    const long long c0 = (chunk0 + lc) * 8;
    float* dst = p.W + (size_t)j * d + c0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      dst[2 * i] = w2[i].x;
      dst[2 * i + 1] = w2[i].y;
    }
  }
}

}  // namespace wpsgd
