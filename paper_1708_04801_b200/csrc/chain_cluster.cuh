// Per-node SGD chains on dense rows, blocked form (see chain_block.cuh for the algebra), with the columns of one
// chain split over the CTAs of a thread-block cluster.
//
// Why: a chain is serial in its samples, so the only way to put more than one SM behind a long chain is to split
// the feature axis. With unequal step counts (the workload of Algorithm 1) one CTA per node leaves the SMs of the
// short chains idle while the longest chain finishes. Here every chain is a cluster of C narrow CTAs and several CTAs
// share an SM: while all chains run, the SM's issue slots are shared; once the short chains are done, the CTAs of the
// long chains have their SMs to themselves.
//
// CTA `rank` of a cluster owns the 16-byte chunks [rank * cpc, (rank + 1) * cpc) of every row. Each CTA has its own
// recurrence warp (warp 0), copy warp (warp 1: bulk asynchronous copies of its column slice of the 8 rows of a future
// block into a ring in shared memory, never multicast) and math warps (the model slice lives in their registers).
// Per block b:
//     math warps    wait for the rows, one pass over them: partial Gram block G_b and partial p_b = X_b w over their
//                   columns (packed two-wide fp32 FMAs), summed over the warp and stored into the partial-sum table
//                   of EVERY CTA of the cluster (distributed shared memory)
//     ------------- cluster barrier (release / acquire) ---------------------------------------------------
//     warp 0        adds the partial sums of all math warps of the cluster, runs the 8-step recurrence, publishes
//                   gamma (every CTA does this redundantly: no second exchange)
//     ------------- CTA barrier -------------------------------------------------------------------------------
//     math warps    w <- w - (1 - a^B) w - sum_m gamma_m x_m from the rows still in shared memory
// The partial-sum tables are double buffered (block parity), so one cluster barrier per block is enough: a CTA can
// be at most one block ahead of its peers. Waits on arriving rows are bounded; a wait that runs out is flagged in
// every CTA of the cluster before the cluster barrier, so all of them leave the loop at the same block.
#pragma once

#include "chain_block.cuh"

namespace wpsgd {

struct ClusterParams {
  BlockParams b;
  int chunks_per_cta;  // cpc: 16-byte chunks of a row owned by one CTA
};

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t cluster_nctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
  return r;
}
// All threads of all CTAs of the cluster; writes before it (also to other CTAs' shared memory) are visible after it.
__device__ __forceinline__ void cluster_barrier() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address of this CTA's shared-memory location `p` in the CTA with the given rank of the cluster.
__device__ __forceinline__ uint32_t map_shared_rank(const void* p, uint32_t rank) {
  const uint32_t a = (uint32_t)__cvta_generic_to_shared(p);
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(rank));
  return r;
}
__device__ __forceinline__ void st_shared_cluster(uint32_t addr, float v) {
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ void st_shared_cluster(uint32_t addr, int v) {
  asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}

constexpr int CL_MAX_SLOTS = 16;  // math warps of a whole cluster

struct ClusterSmem {
  size_t ring, redG, redP, totG, gam, tab, jet, bars, flag, total;
  __host__ __device__ ClusterSmem(int stages, size_t slice_bytes) {
    ring = 0;
    redG = ring + (size_t)stages * BLK_B * slice_bytes;              // [2][slots][32]
    redP = redG + 2 * (size_t)CL_MAX_SLOTS * 32 * sizeof(float);     // [2][slots][8]
    totG = redP + 2 * (size_t)CL_MAX_SLOTS * BLK_B * sizeof(float);  // [32]
    gam = totG + 32 * sizeof(float);                                 // [16]
    tab = gam + 16 * sizeof(float);                                  // [48]
    jet = tab + 3 * 16 * sizeof(float);                              // [8] float4
    bars = jet + 8 * 4 * sizeof(float);                              // [8] barriers
    flag = bars + 8 * sizeof(unsigned long long);
    total = flag + 16;
  }
};

template <typename XT, int R, int LOSS, int MAXMW, int MINB>
__global__ void __launch_bounds__(64 + 32 * MAXMW, MINB) chain_cluster_kernel(const ClusterParams cp) {
  constexpr int V = XVec<XT>::V;
  constexpr int NP = XPairs<XT>::NP;
  constexpr int B = BLK_B;
  extern __shared__ __align__(16) unsigned char smem[];
  const BlockParams& bp = cp.b;
  const ChainParams& p = bp.c;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int math_warps = (blockDim.x >> 5) - 2;
  const int TM = math_warps * 32;
  const int S = bp.stages;
  const uint32_t C = cluster_nctarank(), rank = cluster_ctarank();
  const int j = p.order[blockIdx.x / C];
  const long long n_run = p.n_steps[j];
  const long long d = p.d;
  const long long chunks = d / V;
  const long long chunk0 = (long long)rank * cp.chunks_per_cta;
  const long long chunk_end = chunk0 + cp.chunks_per_cta < chunks ? chunk0 + cp.chunks_per_cta : chunks;
  const int my_chunks = (int)(chunk_end > chunk0 ? chunk_end - chunk0 : 0);
  const size_t slice_bytes = (size_t)cp.chunks_per_cta * 16;  // stride of a staged row slice
  const size_t ld_bytes = (size_t)p.ld * sizeof(XT);
  const ClusterSmem L(S, slice_bytes);
  unsigned char* ring = smem + L.ring;
  float* redG = (float*)(smem + L.redG);
  float* redP = (float*)(smem + L.redP);
  float* totG = (float*)(smem + L.totG);
  float* gam = (float*)(smem + L.gam);  // gamma_0..7, [8] = 1 - a^nv
  float* tab = (float*)(smem + L.tab);  // [0..8] a^k, [16..24] eta / a^{k+1}, [32..40] 1 - a^k
  float4* jets = (float4*)(smem + L.jet);
  unsigned long long* bars = (unsigned long long*)(smem + L.bars);
  volatile int* give_up = (volatile int*)(smem + L.flag);
  const char* shard = (const char*)p.X + (size_t)p.shard_off[j] * ld_bytes + (size_t)chunk0 * 16;
  const float* yshard = p.y + p.shard_off[j];
  const uint32_t* idx = p.idx + p.idx_off[j];
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
  // partial-sum slots that no math warp of the cluster writes stay zero
  for (int i = threadIdx.x; i < 2 * CL_MAX_SLOTS * 32; i += blockDim.x) redG[i] = 0.0f;
  for (int i = threadIdx.x; i < 2 * CL_MAX_SLOTS * B; i += blockDim.x) redP[i] = 0.0f;
  __syncthreads();

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
    cluster_barrier();  // start-up: every CTA of the cluster runs and has cleared its tables

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
      cluster_barrier();  // the partial sums of block b are in every CTA's table
      if (*give_up) break;
      const float* rG = redG + (size_t)(b & 1) * CL_MAX_SLOTS * 32;
      const float* rP = redP + (size_t)(b & 1) * CL_MAX_SLOTS * B;
      float Gs[BLK_PAIRS];  // sc_n G_mn at [n(n-1)/2 + m], m < n
      {
        float gp[CL_MAX_SLOTS];
#pragma unroll
        for (int w = 0; w < CL_MAX_SLOTS; ++w) gp[w] = rG[w * 32 + lane];
#pragma unroll
        for (int h = CL_MAX_SLOTS / 2; h >= 1; h >>= 1)
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
      float pp[CL_MAX_SLOTS];
#pragma unroll
      for (int w = 0; w < CL_MAX_SLOTS; ++w) pp[w] = rP[w * B + n];
#pragma unroll
      for (int h = CL_MAX_SLOTS / 2; h >= 1; h >>= 1)
#pragma unroll
        for (int w = 0; w < h; ++w) pp[w] += pp[w + h];
      const float psum = pp[0];
      float t[B], beta[B];
#pragma unroll
      for (int m = 0; m < B; ++m) t[m] = sc[m] * __shfl_sync(0xffffffffu, psum, m);
      if (LOSS == LOSS_LOGISTIC) {
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
      __syncthreads();  // gamma published
    }
    return;
  }

  if (warp == 1) {
    // =========================== copy warp ==============================================================
    // Lane m < 8 requests this CTA's column slice of row m of a block as one bulk copy; the eight copies complete on
    // the stage's barrier. A stage is refilled after the cluster barrier of the following block: by then every
    // math warp of this CTA has applied the update that was the last read of the stage.
    const uint32_t copy_bytes = (uint32_t)my_chunks * 16u;
    uint32_t id_next = 0u;
    auto peek = [&](long long blk) {
      if (lane < B && blk < nb) id_next = idx[blk * B + lane];
    };
    auto request = [&](long long blk, int stg) {
      if (blk < nb && blk != bp.drop_block && copy_bytes > 0) {
        if (lane == 0) mbar_arrive_expect_tx(&bars[stg], B * copy_bytes);
        __syncwarp();
        if (lane < B)
          bulk_copy_g2s(ring + ((size_t)stg * B + lane) * slice_bytes, shard + (size_t)id_next * ld_bytes, copy_bytes, &bars[stg]);
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
    int st = 0;         // stage of block b - 1
    long long b = 0;
    bool stop = false;
    for (; b < nb; ++b) {
      cluster_barrier();
      if (*give_up) { stop = true; break; }
      if (b >= 1) {
        request(requested, st);
        ++requested;
        peek(requested);
        st = (st + 1 == S) ? 0 : st + 1;
      }
      __syncthreads();
    }
    if (stop && copy_bytes > 0) {
      // leave no copy in flight into this CTA's shared memory: wait (bounded) on the stage of every block that was
      // requested and may not have landed yet
      long long blk = b - 1 > 0 ? b - 1 : 0;
      for (; blk < requested && blk < nb; ++blk)
        if (blk != bp.drop_block) mbar_wait_bounded(&bars[blk % S], (uint32_t)((blk / S) & 1), bp.spin_limit);
    }
    return;
  }

  // ============================= math warps ==============================================================
  const int tm = threadIdx.x - 64;
  const int mw = warp - 2;
  bool act[R];
  float2 w2[R][NP];
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const int lc = r * TM + tm;  // chunk within this CTA's slice
    act[r] = lc < my_chunks;
#pragma unroll
    for (int i = 0; i < NP; ++i) w2[r][i] = make_float2(0.0f, 0.0f);
    if (act[r]) {
      const long long c0 = (chunk0 + lc) * V;
      const float* src = p.resume ? (p.W + (size_t)j * d + c0) : (p.w0 ? p.w0 + c0 : nullptr);
      if (src) {
#pragma unroll
        for (int i = 0; i < NP; ++i) w2[r][i] = make_float2(src[2 * i], src[2 * i + 1]);
      }
    }
  }
  // where this warp's partial sums go in every CTA of the cluster
  const int slot = (int)rank * math_warps + mw;
  cluster_barrier();  // start-up

  int st = 0;
  uint32_t par = 0u;
  for (long long b = 0; b < nb; ++b) {
    if (my_chunks > 0 && !mbar_wait_bounded(&bars[st], par, bp.spin_limit)) {
      set_status(p.status, DEV_TIMEOUT, 1, (long long)blockIdx.x);
      for (uint32_t rr = 0; rr < C; ++rr) st_shared_cluster(map_shared_rank((const void*)give_up, rr), 1);
    }
    const unsigned char* stage = ring + (size_t)st * B * slice_bytes;
    // ---- G_b and p_b partials over this thread's columns ------------------------------------------------------
    float2 acc2[BLK_PAIRS], accp2[B];
#pragma unroll
    for (int i = 0; i < BLK_PAIRS; ++i) acc2[i] = make_float2(0.0f, 0.0f);
#pragma unroll
    for (int m = 0; m < B; ++m) accp2[m] = make_float2(0.0f, 0.0f);
#pragma unroll
    for (int r = 0; r < R; ++r) {
      if (act[r]) {
        uint4 raw[B];
#pragma unroll
        for (int m = 0; m < B; ++m) raw[m] = *(const uint4*)(stage + (size_t)m * slice_bytes + (size_t)(r * TM + tm) * 16);
#pragma unroll
        for (int i = 0; i < NP; ++i) {
          float2 x2[B];
#pragma unroll
          for (int m = 0; m < B; ++m) x2[m] = XPairs<XT>::get(raw[m], i);
#pragma unroll
          for (int n2 = 1; n2 < B; ++n2)
#pragma unroll
            for (int m = 0; m < n2; ++m) acc2[n2 * (n2 - 1) / 2 + m] = __ffma2_rn(x2[m], x2[n2], acc2[n2 * (n2 - 1) / 2 + m]);
#pragma unroll
          for (int m = 0; m < B; ++m) accp2[m] = __ffma2_rn(w2[r][i], x2[m], accp2[m]);
        }
      }
    }
    float acc[32], accp[B];
#pragma unroll
    for (int i = 0; i < BLK_PAIRS; ++i) acc[i] = acc2[i].x + acc2[i].y;
#pragma unroll
    for (int i = BLK_PAIRS; i < 32; ++i) acc[i] = 0.0f;
#pragma unroll
    for (int m = 0; m < B; ++m) accp[m] = accp2[m].x + accp2[m].y;
    const float gtot = warp_transpose_sum32(acc);  // lane l: Gram entry l over the warp's columns
    const float ptot = warp_transpose_sum8(accp);  // every lane: p_{lane >> 2} over the warp's columns
    {
      float* dg = redG + ((size_t)(b & 1) * CL_MAX_SLOTS + slot) * 32 + lane;
      float* dp = redP + ((size_t)(b & 1) * CL_MAX_SLOTS + slot) * B + (lane >> 2);
      for (uint32_t rr = 0; rr < C; ++rr) {
        st_shared_cluster(map_shared_rank(dg, rr), gtot);
        if ((lane & 3) == 0) st_shared_cluster(map_shared_rank(dp, rr), ptot);
      }
    }
    cluster_barrier();
    if (*give_up) break;
    __syncthreads();  // gamma_b is in gam
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
      for (int r = 0; r < R; ++r) {
        if (act[r]) {
          uint4 raw[B];
#pragma unroll
          for (int m = 0; m < B; ++m) raw[m] = *(const uint4*)(stage + (size_t)m * slice_bytes + (size_t)(r * TM + tm) * 16);
#pragma unroll
          for (int i = 0; i < NP; ++i) {
            float2 wv = __ffma2_rn(ndl2, w2[r][i], w2[r][i]);
#pragma unroll
            for (int m = 0; m < B; ++m) wv = __ffma2_rn(ngm2[m], XPairs<XT>::get(raw[m], i), wv);
            w2[r][i] = wv;
          }
        }
      }
    }
    if (++st == S) { st = 0; par ^= 1u; }
  }

#pragma unroll
  for (int r = 0; r < R; ++r) {
    if (act[r]) {
      const long long c0 = (chunk0 + r * TM + tm) * V;
      float* dst = p.W + (size_t)j * d + c0;
#pragma unroll
      for (int i = 0; i < NP; ++i) {
        dst[2 * i] = w2[r][i].x;
        dst[2 * i + 1] = w2[r][i].y;
      }
    }
  }
}

}  // namespace wpsgd
