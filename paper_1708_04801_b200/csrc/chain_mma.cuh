// Per-node SGD chains on dense bf16 rows, blocked form (see chain_block.cuh for the algebra), with the Gram block
// and the margins of a block from the warp-level tensor-core instruction and the columns of a chain split over the
// CTAs of a thread-block cluster.
//
// What a block of B = 8 samples needs before its scalar recurrence is G = X_b X_b^T (8 x 8) and p = X_b w (8): one
// product [X_b ; w] X_b^T of an (8 + 1) x d by a d x 8 matrix. The rows are bf16, so their products are exact in fp32
// and the tensor core accumulates them in fp32. The model is fp32; it is written as w = w_hi + w_mid + w_lo with three
// bf16 terms (8 + 8 + 8 mantissa bits, each remainder exact), which enter the product as three more rows. One
// mma.m16n8k16 per 16 columns then gives, in its 16 x 8 accumulator, rows 0..7 = G and rows 8..10 = the three parts
// of p: no widening of the rows, no FMA per column pair, no cross-lane reduction (the instruction sums over its 16
// columns, the accumulator over the warp's 256). Only the update w <- w - (1 - a^B) w - sum_m gamma_m x_m stays on
// the fp32 pipes (packed two-wide FMAs), followed by re-splitting the thread's 8 model values into the three bf16 rows.
//
// Layout. CTA `rank` of a cluster of C owns the 16-byte chunks [rank * cpc, (rank + 1) * cpc) of every row. A lane
// owns NPL pairs of consecutive columns (NPL = 4: one 16-byte chunk, 8 math warps cover 2048 columns, the default;
// NPL = 2: half a chunk, 16 math warps, which halves the instruction stream of a math warp but doubles the partial
// sums the recurrence warp adds, and measured slower), math warp mw the 32 consecutive lane units from 32 mw; the
// model values live in registers.
// Warp 0 runs the recurrence, warp 1 requests rows (bulk asynchronous copies into a ring of stages, one barrier per
// stage, never multicast). Staged rows and the three model rows have a stride of slice + 16 bytes, which keeps the
// 8 x 8 tile loads (ldmatrix) free of bank conflicts; bytes beyond a CTA's slice stay zero.
//
// Exchange inside the cluster. Every math warp sends its 64 + 24 accumulator values to the partial-sum table of
// every CTA of the cluster with st.async (a store to distributed shared memory that reports its bytes to a barrier
// of the destination CTA). The recurrence warp of each CTA arms that barrier with the byte count of all math warps
// of the cluster and waits for it (bounded), adds the partial sums, runs the recurrence and publishes gamma in its
// own CTA: every CTA does this redundantly, so there is one exchange per block and no cluster-wide barrier inside
// the loop. Tables and barriers are double buffered by block parity; a CTA cannot receive block b + 2 before it has
// consumed block b, because its peers need its own block b + 1 first.
//
// Leaving. A wait that runs out (rows or partial sums) sets the status word and the give-up flag of every CTA of
// the cluster. The recurrence warp samples the flag once per block and publishes the decision with gamma, so all
// warps of a CTA leave at the same block; every thread then passes one final cluster barrier, so no CTA exits while
// a peer may still store into its shared memory.
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


constexpr int MMA_SLOTS = 16;    // math warps of a whole cluster (one 16-byte chunk per lane); twice that with half chunks
constexpr int MMA_G_VALS = 64;   // accumulator rows 0..7
constexpr int MMA_P_VALS = 32;   // accumulator rows 8..10 (24 used)
constexpr uint32_t MMA_SLOT_BYTES = (64 + 24) * sizeof(float);  // what one math warp sends to one CTA per block

struct MmaSmem {
  size_t row_stride, ring, w3, redG, redP, totG, gam, tab, jet, bars, pbar, flag, total;
  __host__ __device__ MmaSmem(int stages, size_t slice_bytes, int slots) {
    row_stride = slice_bytes + 16;
    ring = 0;
    w3 = ring + (size_t)stages * BLK_B * row_stride;                // w_hi, w_mid, w_lo, one zero row
    redG = w3 + 4 * row_stride;                                     // [2][slots][64]
    redP = redG + 2 * (size_t)slots * MMA_G_VALS * sizeof(float);  // [2][slots][32]
    totG = redP + 2 * (size_t)slots * MMA_P_VALS * sizeof(float);  // [64] G, [32] parts of p
    gam = totG + 96 * sizeof(float);                                // gamma_0..7, 1 - a^nv, stop
    tab = gam + 16 * sizeof(float);                                 // [48]
    jet = tab + 3 * 16 * sizeof(float);                             // [8] float4
    bars = jet + 8 * 4 * sizeof(float);                             // ring barriers [8]
    pbar = bars + 8 * sizeof(unsigned long long);                   // partial-sum barriers [2]
    flag = pbar + 2 * sizeof(unsigned long long);
    total = flag + 16;
  }
};

// 8-byte store into the shared memory of a CTA of the cluster; its 8 bytes are counted on that CTA's barrier `mbar`
// (both addresses in the shared::cluster window of the same CTA).
__device__ __forceinline__ void st_async_f32x2(uint32_t addr, float a, float b, uint32_t mbar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v2.f32 [%0], {%1, %2}, [%3];" ::"r"(addr),
               "f"(a), "f"(b), "r"(mbar)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(unsigned long long* bar, uint32_t parity) {
  const uint32_t a = (uint32_t)__cvta_generic_to_shared(bar);
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(a), "r"(parity)
      : "memory");
  return ok != 0;
}
// Later asynchronous-proxy writes (bulk copies) to shared memory are ordered after this thread's earlier stores.
__device__ __forceinline__ void fence_proxy_async_shared() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Two fp32 -> packed bf16 (round to nearest even); the low half holds `lo`, the high half `hi`.
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

template <int LOSS, int NPL>
__global__ void __launch_bounds__(NPL == 4 ? 64 + 32 * 8 : 64 + 32 * 16, 1) chain_mma_kernel(const ClusterParams cp) {
  constexpr int B = BLK_B;
  constexpr int LB = NPL * 4;                     // bytes of a row per lane
  constexpr int KS = LB;                          // 16-column steps per warp (32 lanes x LB bytes / 32 bytes)
  constexpr int SLOTS = MMA_SLOTS * (4 / NPL);    // partial-sum slots of the cluster
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
  const MmaSmem L(S, slice_bytes, SLOTS);
  const size_t row_stride = L.row_stride;
  unsigned char* ring = smem + L.ring;
  unsigned char* w3 = smem + L.w3;
  float* redG = (float*)(smem + L.redG);
  float* redP = (float*)(smem + L.redP);
  float* totG = (float*)(smem + L.totG);
  float* gam = (float*)(smem + L.gam);
  float* tab = (float*)(smem + L.tab);  // [0..8] a^k, [16..24] eta / a^{k+1}, [32..40] 1 - a^k
  float4* jets = (float4*)(smem + L.jet);
  unsigned long long* bars = (unsigned long long*)(smem + L.bars);
  unsigned long long* pbar = (unsigned long long*)(smem + L.pbar);
  volatile int* give_up = (volatile int*)(smem + L.flag);
  const char* shard = (const char*)p.X + (size_t)p.shard_off[j] * ld_bytes + (size_t)chunk0 * 16;
  const float* yshard = p.y + p.shard_off[j];
  const uint32_t* idx = p.idx + p.idx_off[j];
  const long long nb = (n_run + B - 1) / B;

  // ---- set-up: tables, barriers, zeroed ring / model rows / partial-sum tables ------------------------------------
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
    mbar_init(&pbar[0], 1);
    mbar_init(&pbar[1], 1);
    *give_up = 0;
    mbar_fence_init();
  }
  {
    // everything from the ring up to the end of the partial-sum tables starts at zero: columns beyond a slice, the
    // zero row of the model rows and the table slots that no math warp writes are never written later
    uint4* z = (uint4*)smem;
    const int n16 = (int)(L.totG / 16);
    for (int i = threadIdx.x; i < n16; i += blockDim.x) z[i] = make_uint4(0u, 0u, 0u, 0u);
  }
  fence_proxy_async_shared();
  __syncthreads();

  if (warp == 0) {
    // =========================== recurrence warp ========================================================
    const int n = lane & (B - 1);
    float y_nxt = 0.0f;
    uint32_t id_nxt = 0u;
    if (nb > 0) y_nxt = yshard[idx[n]];
    if (nb > 1) id_nxt = idx[B + n];
    float apw[B], cfac[B];
#pragma unroll
    for (int m = 0; m < B; ++m) { apw[m] = tab[m]; cfac[m] = tab[16 + m]; }
    const bool decaying = p.sched == LR_INV_SQRT;
    const long long first_j = p.first ? p.first[j] : 0;
    const uint32_t expect_bytes = C * (uint32_t)math_warps * MMA_SLOT_BYTES;
    cluster_barrier();  // start-up: every CTA of the cluster runs and has set up its shared memory

    for (long long b = 0; b < nb; ++b) {
      const int nv = (int)((n_run - b * B) < (long long)B ? (n_run - b * B) : (long long)B);
      const int q = (int)(b & 1);
      if (lane == 0) mbar_arrive_expect_tx(&pbar[q], expect_bytes);
      const float y_cur = y_nxt;
      if (b + 1 < nb) y_nxt = yshard[id_nxt];
      if (b + 2 < nb) id_nxt = idx[(b + 2) * B + n];
      float a_nv = tab[nv], dl_nv = tab[32 + nv], apw_own = tab[n];
      if (decaying) decaying_block_tables<B>((double)p.eta0, (double)p.lambda, first_j + b * B, nv, apw, cfac, apw_own, a_nv, dl_nv);
      float yv[B], sc[B], cf[B];
#pragma unroll
      for (int m = 0; m < B; ++m) yv[m] = __shfl_sync(0xffffffffu, y_cur, m);
      block8_constants<LOSS>(yv, apw, cfac, nv, sc, cf);
      // ---- wait (bounded) for the partial sums of block b from every math warp of the cluster ------------------
      {
        const uint32_t parity = (uint32_t)((b >> 1) & 1);
        bool landed = false;
        for (long long i = 0; i < bp.spin_limit; ++i) {
          if (mbar_try_wait_cluster(&pbar[q], parity)) { landed = true; break; }
          if (*give_up) break;
        }
        if (!landed && !*give_up) {
          set_status(p.status, DEV_TIMEOUT, 2, (long long)blockIdx.x);
          for (uint32_t rr = 0; rr < C; ++rr) st_shared_cluster(map_shared_rank((const void*)give_up, rr), 1);
        }
      }
      const int stop = *give_up;
      const float* rG = redG + (size_t)q * SLOTS * MMA_G_VALS;
      const float* rP = redP + (size_t)q * SLOTS * MMA_P_VALS;
      float Gs[BLK_PAIRS];  // sc_n G_mn at [n(n-1)/2 + m], m < n
      float psum;           // lane l: p of sample l & 7
      {
        // one pass over the slots with 16-byte loads: lanes 0..15 add four consecutive entries of G each, lanes
        // 16..23 four of the parts of p
        if (lane < 24) {
          const float* base = lane < 16 ? rG + lane * 4 : rP + (lane & 7) * 4;
          const int stride = lane < 16 ? MMA_G_VALS : MMA_P_VALS;
          float4 s4 = *(const float4*)base;
#pragma unroll
          for (int w = 1; w < SLOTS; ++w) {
            const float4 v = *(const float4*)(base + w * stride);
            s4.x += v.x; s4.y += v.y; s4.z += v.z; s4.w += v.w;
          }
          ((float4*)totG)[lane] = s4;
        }
        __syncwarp();
#pragma unroll
        for (int n2 = 1; n2 < B; ++n2) {
          const float4 lo = *(const float4*)&totG[n2 * 8], hi = *(const float4*)&totG[n2 * 8 + 4];
          const float row[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
#pragma unroll
          for (int m = 0; m < n2; ++m) Gs[n2 * (n2 - 1) / 2 + m] = row[m] * sc[n2];
        }
        // rows 8..10 of the accumulator: w_hi . x_n, w_mid . x_n, w_lo . x_n; small terms first
        psum = (totG[64 + 16 + n] + totG[64 + 8 + n]) + totG[64 + n];
        __syncwarp();
      }
      float t[B], beta[B];
#pragma unroll
      for (int m = 0; m < B; ++m) t[m] = sc[m] * __shfl_sync(0xffffffffu, psum, m);
      block8_recurrence<LOSS>(t, Gs, cf, yv, y_cur * apw_own * 1.4426950408889634f * psum, jets, beta);
      // gamma_m = eta g_m a^{nv-1-m} = beta_m a^{nv}; [8] = 1 - a^nv; [9] = leave after this block
      float mine = dl_nv;
#pragma unroll
      for (int m = 0; m < B; ++m)
        if (lane == m) mine = beta[m] * a_nv;
      if (lane == B + 1) mine = stop ? 1.0f : 0.0f;
      if (lane <= B + 1) gam[lane] = mine;
      __syncthreads();  // gamma and the decision published
      if (stop) break;
    }
    cluster_barrier();  // nobody exits while a peer may still store into its shared memory
    return;
  }

  if (warp == 1) {
    // =========================== copy warp ==============================================================
    // Lane m < 8 requests this CTA's column slice of row m of a block as one bulk copy; the eight copies complete on
    // the stage's barrier. A stage is refilled right after the CTA barrier of its block: by then every math warp of
    // this CTA has run the tensor-core pass over it and holds its own columns of the rows in registers.
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
          bulk_copy_g2s(ring + ((size_t)stg * B + lane) * row_stride, shard + (size_t)id_next * ld_bytes, copy_bytes, &bars[stg]);
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
    int st = 0;         // stage of block b
    long long b = 0;
    bool stop = false;
    for (; b < nb; ++b) {
      __syncthreads();
      if (gam[B + 1] != 0.0f) { stop = true; break; }
      request(requested, st);
      ++requested;
      peek(requested);
      st = (st + 1 == S) ? 0 : st + 1;
    }
    if (stop && copy_bytes > 0) {
      // leave no copy in flight into this CTA's shared memory: wait (bounded) on the stage of every block that was
      // requested and may not have landed yet
      long long blk = b;
      for (; blk < requested && blk < nb; ++blk)
        if (blk != bp.drop_block) mbar_wait_bounded(&bars[blk % S], (uint32_t)((blk / S) & 1), bp.spin_limit);
    }
    cluster_barrier();
    return;
  }

  // ============================= math warps ==============================================================
  const int mw = warp - 2;
  const int lc = mw * 32 + lane;  // this thread's unit (LB bytes of a row) within the CTA's slice
  const int my_units = my_chunks * (16 / LB);
  const bool act = lc < my_units;
  const int warp_units = my_units - mw * 32 < 0 ? 0 : (my_units - mw * 32 > 32 ? 32 : my_units - mw * 32);
  const int ksteps = (warp_units * LB + 31) / 32;  // 16 columns (32 bytes) per tensor-core instruction
  float2 w2[NPL];
#pragma unroll
  for (int i = 0; i < NPL; ++i) w2[i] = make_float2(0.0f, 0.0f);
  if (act) {
    const long long c0 = chunk0 * 8 + (long long)lc * (2 * NPL);
    const float* src = p.resume ? (p.W + (size_t)j * d + c0) : (p.w0 ? p.w0 + c0 : nullptr);
    if (src) {
#pragma unroll
      for (int i = 0; i < NPL; ++i) w2[i] = make_float2(src[2 * i], src[2 * i + 1]);
    }
  }
  // LB bytes of shared memory as NPL words
  auto load_words = [&](const unsigned char* ptr, uint32_t (&wd)[NPL]) __attribute__((always_inline)) {
    if (NPL == 4) {
      const uint4 v = *(const uint4*)ptr;
      wd[0] = v.x; wd[1] = v.y; wd[NPL - 2] = v.z; wd[NPL - 1] = v.w;
    } else {
      const uint2 v = *(const uint2*)ptr;
      wd[0] = v.x; wd[1] = v.y;
    }
  };
  auto store_words = [&](unsigned char* ptr, const uint32_t (&wd)[NPL]) __attribute__((always_inline)) {
    if (NPL == 4) *(uint4*)ptr = make_uint4(wd[0], wd[1], wd[NPL - 2], wd[NPL - 1]);
    else *(uint2*)ptr = make_uint2(wd[0], wd[1]);
  };
  // the thread's model values as three bf16 rows: w = hi + mid + lo (each remainder is exact in fp32)
  auto publish_model = [&]() __attribute__((always_inline)) {
    if (act) {
      uint32_t hi[NPL], mid[NPL], lo[NPL];
#pragma unroll
      for (int i = 0; i < NPL; ++i) {
        hi[i] = pack_bf16x2(w2[i].x, w2[i].y);
        const float rx = w2[i].x - __uint_as_float(hi[i] << 16), ry = w2[i].y - __uint_as_float(hi[i] & 0xffff0000u);
        mid[i] = pack_bf16x2(rx, ry);
        const float sx = rx - __uint_as_float(mid[i] << 16), sy = ry - __uint_as_float(mid[i] & 0xffff0000u);
        lo[i] = pack_bf16x2(sx, sy);
      }
      store_words(w3 + 0 * row_stride + (size_t)lc * LB, hi);
      store_words(w3 + 1 * row_stride + (size_t)lc * LB, mid);
      store_words(w3 + 2 * row_stride + (size_t)lc * LB, lo);
    }
    __syncwarp();
  };
  publish_model();
  // tile addresses of the tensor-core operand loads: lanes 8i..8i+7 give the 8 row addresses of tile i; tiles 0 and 2
  // are the staged rows (columns +0 and +8), tiles 1 and 3 the model rows (hi, mid, lo, then the zero row)
  const int tile = lane >> 3, trow = lane & 7;
  const size_t tile_col_bytes = (size_t)mw * (32 * LB) + (size_t)(tile >> 1) * 16;
  const size_t x_off = (size_t)trow * row_stride + tile_col_bytes;
  const unsigned char* w_src = w3 + (size_t)(trow < 3 ? trow : 3) * row_stride + tile_col_bytes;
  const int slot = (int)rank * math_warps + mw;
  // shared-memory window of every CTA of the cluster (the same offsets apply inside each window)
  const uint32_t own_base = (uint32_t)__cvta_generic_to_shared(smem);
  uint32_t peer_base[8];
#pragma unroll
  for (int rr = 0; rr < 8; ++rr) peer_base[rr] = map_shared_rank(smem, (uint32_t)rr < C ? (uint32_t)rr : rank);
  cluster_barrier();  // start-up

  int st = 0;
  uint32_t par = 0u;
  for (long long b = 0; b < nb; ++b) {
    if (my_chunks > 0 && !mbar_wait_bounded(&bars[st], par, bp.spin_limit)) {
      set_status(p.status, DEV_TIMEOUT, 1, (long long)blockIdx.x);
      for (uint32_t rr = 0; rr < C; ++rr) st_shared_cluster(map_shared_rank((const void*)give_up, rr), 1);
    }
    const unsigned char* stage = ring + (size_t)st * B * row_stride;
    // ---- [G_b ; p_b parts] over this warp's columns ------------------------------------------------------------
    // four independent accumulators (a dependent mma.sync takes about 20 cycles); the operand tiles are loaded four
    // at a time
    constexpr int NACC = 4;
    float acc[NACC][4];
#pragma unroll
    for (int a = 0; a < NACC; ++a)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[a][e] = 0.0f;
    {
      const unsigned char* src = (tile & 1) ? w_src : stage + x_off;
#pragma unroll
      for (int round = 0; round < KS / 4; ++round) {
        uint32_t q[4][4];
#pragma unroll
        for (int a = 0; a < 4; ++a)
          if (round * 4 + a < ksteps) ldmatrix_x4(q[a], src + (size_t)(round * 4 + a) * 32);
#pragma unroll
        for (int a = 0; a < 4; ++a)
          if (round * 4 + a < ksteps) mma_bf16_m16n8k16(acc[a], q[a][0], q[a][1], q[a][2], q[a][3], q[a][0], q[a][2]);
      }
    }
#pragma unroll
    for (int h = NACC / 2; h >= 1; h >>= 1)
#pragma unroll
      for (int a = 0; a < h; ++a)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[a][e] += acc[a + h][e];
    {
      // accumulator rows 0..7: lane l holds G[l / 4][2 (l % 4) .. +1]; rows 8..10 (lanes 0..11): the parts of p
      const int q = (int)(b & 1);
      const uint32_t og = (uint32_t)__cvta_generic_to_shared(redG + ((size_t)q * SLOTS + slot) * MMA_G_VALS + lane * 2) - own_base;
      const uint32_t op = (uint32_t)__cvta_generic_to_shared(redP + ((size_t)q * SLOTS + slot) * MMA_P_VALS + lane * 2) - own_base;
      const uint32_t ob = (uint32_t)__cvta_generic_to_shared(&pbar[q]) - own_base;
#pragma unroll
      for (int rr = 0; rr < 8; ++rr) {
        if ((uint32_t)rr < C) {
          st_async_f32x2(peer_base[rr] + og, acc[0][0], acc[0][1], peer_base[rr] + ob);
          if (lane < 12) st_async_f32x2(peer_base[rr] + op, acc[0][2], acc[0][3], peer_base[rr] + ob);
        }
      }
    }
    // this thread's columns of the 8 rows, for the update: afterwards the stage can be refilled
    uint32_t raw[B][NPL];
#pragma unroll
    for (int m = 0; m < B; ++m) {
#pragma unroll
      for (int i = 0; i < NPL; ++i) raw[m][i] = 0u;
      if (act) load_words(stage + (size_t)m * row_stride + (size_t)lc * LB, raw[m]);
    }
    __syncthreads();  // gamma_b and the decision are in gam; every math warp is done with the stage
    if (gam[B + 1] != 0.0f) break;
    // ---- w <- w - (1 - a^nv) w - sum_m gamma_m x_m, then the model rows again -----------------------------------------
    if (act) {
      float2 ngm2[B];
#pragma unroll
      for (int m = 0; m < B; ++m) {
        const float g = -gam[m];
        ngm2[m] = make_float2(g, g);
      }
      const float ndl = -gam[B];
      const float2 ndl2 = make_float2(ndl, ndl);
#pragma unroll
      for (int i = 0; i < NPL; ++i) {
        float2 wv = __ffma2_rn(ndl2, w2[i], w2[i]);
#pragma unroll
        for (int m = 0; m < B; ++m)
          wv = __ffma2_rn(ngm2[m], make_float2(__uint_as_float(raw[m][i] << 16), __uint_as_float(raw[m][i] & 0xffff0000u)), wv);
        w2[i] = wv;
      }
    }
    publish_model();
    if (++st == S) { st = 0; par ^= 1u; }
  }
  cluster_barrier();

  if (act) {
    const long long c0 = chunk0 * 8 + (long long)lc * (2 * NPL);
    float* dst = p.W + (size_t)j * d + c0;
#pragma unroll
    for (int i = 0; i < NPL; ++i) {
      dst[2 * i] = w2[i].x;
      dst[2 * i + 1] = w2[i].y;
    }
  }
}

}  // namespace wpsgd
