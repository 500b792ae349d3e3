// Per-node SGD chains on dense bf16 rows, blocked form with B = 16 samples per block (the algebra is that of
// chain_block.cuh; the layout, the cluster exchange and the leaving protocol are those of chain_mma.cuh).
//
// Why 16. A block costs a fixed string of hand-offs whatever its size (partial sums out to the cluster, their
// arrival, the recurrence warp, gamma back through a CTA barrier, the model split again for the tensor cores), and
// with 8 samples those hand-offs are the larger half of the block's time. With 16 samples they are paid half as
// often; the price is a 16 x 16 Gram block and a 16-step recurrence.
//
// Tensor-core pass. Per 16 columns the 16 staged rows X are one A tile (ldmatrix.x4) whose registers are, read the
// other way, the B tiles of the same rows (samples 0..7 and 8..15), and the three bf16 rows of the model
// (w = w_hi + w_mid + w_lo, see chain_mma.cuh) are a third B tile (ldmatrix.x2). Three mma.m16n8k16 then give
//     D0 = X X_{0..7}^T    (16 x 8)   Gram entries G[n][m], m < 8
//     D1 = X X_{8..15}^T   (16 x 8)   rows 8..15: G[n][m], 8 <= m
//     D2 = X [w_hi w_mid w_lo 0 ..]^T (16 x 8)   columns 0..2: the three parts of p_n = w . x_n
// with exact bf16 products and fp32 accumulation. 48 bytes of operand reads per sample and 16 columns instead of 64.
//
// What bounds a block. On this part a warp issues one mma.m16n8k16 about every 25 to 30 cycles whatever the number of
// independent accumulators (the tensor pipe itself is busy 8 cycles per step), so the 48 steps of a warp's pass take
// 1100 to 1350 cycles and only more warps would shorten them; with eight math warps, the recurrence warp and the copy
// warp the register file (allocated four warps at a time: 384 threads x 168 registers) has no room for more warps of
// this size. Measured on one chain of d = 4096 (cycles per block; this kernel: 3860):
//   - Gram part (D0, D1) of block b + 1 formed while the recurrence warp works on block b, operand registers kept for
//     the margin part: 3990. The 16 dependent margin steps alone take 750 to 1000 cycles, the recurrence warp's few
//     loads queue behind eight warps' operand loads in the shared-memory pipe (its sums: 975 cycles instead of 100), and
//     with the operand registers kept the update has to read its rows from shared memory again (850 instead of 400).
//   - Margins in fp32 from the row registers (no bf16 copy of the model), Gram part two blocks ahead: 4390 to 4620. The
//     rows are then unpacked twice per block on the integer pipe, and update and margin pass take 1200 cycles each.
//   - Gram part by two warps of their own (they fit the register file for free): 4620. One warp needs 4200 cycles for the
//     128 steps of half the columns, longer than a block.
//   - Ten math warps of 26 chunks instead of eight of 32 (the register allocation is the same): 4560.
//   - gamma of the first eight samples handed to the math warps while the other eight steps run: 3890 (no gain).
//
// The recurrence warp runs the 16 steps as two groups of 8: within a group every lane steps redundantly on registers (no
// shuffle in the dependent chain, as in the 8-sample kernels); between the groups the 8 x 8 cross block is applied one
// row per lane and gathered with eight shuffles. The logistic loss runs each group through the 8-sample recurrence with
// its factor expanded around the group's margins (block8_recurrence).
#pragma once

#include "chain_mma.cuh"

namespace wpsgd {

constexpr int M16_B = 16;
constexpr int M16_PAIRS = M16_B * (M16_B - 1) / 2;  // 120
constexpr int M16_SLOT_FLOATS = 256;   // D0 [16][8] | D1 rows 8..15 [8][8] | p parts [16][4]
constexpr uint32_t M16_SLOT_BYTES = M16_SLOT_FLOATS * sizeof(float);
constexpr int M16_SLOTS = 8;           // one slot per CTA of the cluster
constexpr int M16_WARPS = 8;           // math warps of a CTA

struct Mma16Smem {
  size_t row_stride, ring, w3, red, part, tot, gam, tab, jet, bars, pbar, flag, total;
  __host__ __device__ Mma16Smem(int stages, size_t slice_bytes, int nbuf) {
    row_stride = slice_bytes + 16;
    ring = 0;
    w3 = ring + (size_t)stages * M16_B * row_stride;                 // w_hi, w_mid, w_lo, one zero row
    red = w3 + 4 * row_stride;                                       // [nbuf][slots][256] partial sums
    part = red + (size_t)nbuf * M16_SLOTS * M16_SLOT_FLOATS * sizeof(float);  // [math warps][256] this CTA's partial sums
    tot = part + (size_t)M16_WARPS * M16_SLOT_FLOATS * sizeof(float);      // [256] sums over the slots
    gam = tot + M16_SLOT_FLOATS * sizeof(float);                     // gamma_0..15, 1 - a^nv, stop
    tab = gam + 32 * sizeof(float);                                  // [3][32]
    jet = tab + 3 * 32 * sizeof(float);                              // 8 x (s, s', s''/2, s'''/6) of the logistic factor
    bars = jet + 8 * 4 * sizeof(float);                             // ring barriers [8]
    pbar = bars + 8 * sizeof(unsigned long long);                    // partial-sum barriers [nbuf <= 4]
    flag = pbar + 4 * sizeof(unsigned long long);
    total = flag + 16;
  }
};

// 16-byte store into the shared memory of a CTA of the cluster, counted on that CTA's barrier `mbar`
__device__ __forceinline__ void st_async_f32x4(uint32_t addr, float4 v, uint32_t mbar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.f32 [%0], {%1, %2, %3, %4}, [%5];" ::"r"(addr),
               "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w), "r"(mbar)
               : "memory");
}

__device__ __forceinline__ void ldmatrix_x2(uint32_t (&r)[2], const void* smem_ptr) {
  const uint32_t a = (uint32_t)__cvta_generic_to_shared(smem_ptr);
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "r"(a) : "memory");
}

// XT = __nv_bfloat16: the tensor-core form described above. XT = float: the same blocks, cluster exchange and recurrence
// for fp32 rows with the Gram block and the margins on the fp32 pipes (see the math warps' second part below); there
// the Gram part of block b + 1 is formed while the recurrence warp works on block b, so the sums exist three times.
template <int LOSS, typename XT>
__global__ void __launch_bounds__(64 + 32 * 8, 1) chain_mma16_kernel(const ClusterParams cp) {
  constexpr int B = M16_B;
  constexpr bool F32 = sizeof(XT) == 4;
  constexpr int NBUF = F32 ? 3 : 2;
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
  const long long chunks = d / (16 / (long long)sizeof(XT));  // 16-byte chunks of a row
  const long long chunk0 = (long long)rank * cp.chunks_per_cta;
  const long long chunk_end = chunk0 + cp.chunks_per_cta < chunks ? chunk0 + cp.chunks_per_cta : chunks;
  const int my_chunks = (int)(chunk_end > chunk0 ? chunk_end - chunk0 : 0);
  const size_t slice_bytes = (size_t)cp.chunks_per_cta * 16;
  const size_t ld_bytes = (size_t)p.ld * sizeof(XT);
  const Mma16Smem L(S, slice_bytes, NBUF);
  const size_t row_stride = L.row_stride;
  unsigned char* ring = smem + L.ring;
  unsigned char* w3 = smem + L.w3;
  float* red = (float*)(smem + L.red);
  float* part = (float*)(smem + L.part);
  float* tot = (float*)(smem + L.tot);
  float* gam = (float*)(smem + L.gam);   // [0..15] gamma, [16] = 1 - a^nv, [17] = leave after this block
  float4* jets = (float4*)(smem + L.jet);
  float* tab = (float*)(smem + L.tab);   // [0..16] a^k, [32..48] eta / a^{k+1}, [64..80] 1 - a^k
  unsigned long long* bars = (unsigned long long*)(smem + L.bars);
  unsigned long long* pbar = (unsigned long long*)(smem + L.pbar);
  volatile int* give_up = (volatile int*)(smem + L.flag);
  const char* shard = (const char*)p.X + (size_t)p.shard_off[j] * ld_bytes + (size_t)chunk0 * 16;
  const float* yshard = p.y + p.shard_off[j];
  const uint32_t* idx = p.idx + p.idx_off[j];  // padded to a multiple of 64 entries, all valid rows
  const long long nb = (n_run + B - 1) / B;
  const int consumed_threads = (math_warps + 1) * 32;  // math warps arrive, the copy warp waits: named barrier 2
  const int math_threads = math_warps * 32;

  // ---- set-up: tables, barriers, zeroed ring / model rows / partial-sum tables ------------------------------------
  if (threadIdx.x <= B) {  // power tables in fp64, rounded once
    const double a = 1.0 - bp.eta_lambda;
    double pw = 1.0;
    for (int k = 0; k < (int)threadIdx.x; ++k) pw *= a;
    tab[threadIdx.x] = (float)pw;
    tab[32 + threadIdx.x] = (float)((double)p.eta0 / (pw * a));
    tab[64 + threadIdx.x] = (float)(1.0 - pw);
  }
  if (threadIdx.x == 32) {
    for (int s = 0; s < S; ++s) mbar_init(&bars[s], 1);
    for (int i = 0; i < NBUF; ++i) mbar_init(&pbar[i], 1);
    *give_up = 0;
    mbar_fence_init();
  }
  {
    // everything from the ring up to the end of the partial-sum tables starts at zero: columns beyond a slice, the
    // zero row of the model rows and the table slots that no math warp writes are never written later
    uint4* z = (uint4*)smem;
    const int n16 = (int)(L.tot / 16);
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
    const uint32_t expect_bytes = C * M16_SLOT_BYTES;
    const bool decaying = p.sched == LR_INV_SQRT;
    const long long first_j = p.first ? p.first[j] : 0;
    cluster_barrier();  // start-up: every CTA of the cluster runs and has set up its shared memory

    for (long long b = 0; b < nb; ++b) {
      const int nv = (int)((n_run - b * B) < (long long)B ? (n_run - b * B) : (long long)B);
      const int q = (int)(b % NBUF);
      if (lane == 0) mbar_arrive_expect_tx(&pbar[q], expect_bytes);
      const float y_cur = y_nxt;  // lane l: label of sample l & 15
      if (b + 1 < nb) y_nxt = yshard[id_nxt];
      if (b + 2 < nb) id_nxt = idx[(b + 2) * B + n];
      float a_nv = tab[nv], dl_nv = tab[64 + nv];
      float apw[B], cfac[B];
      float apw_own = tab[n];  // A of this lane's own sample (lane & 15)
      if (decaying) {
        decaying_block_tables<B>((double)p.eta0, (double)p.lambda, first_j + b * B, nv, apw, cfac, apw_own, a_nv, dl_nv);
      } else {
#pragma unroll
        for (int m = 0; m < B; ++m) { apw[m] = tab[m]; cfac[m] = tab[32 + m]; }
      }
      // ---- wait (bounded) for the partial sums of block b from every math warp of the cluster ------------------
      {
        const uint32_t parity = (uint32_t)((b / NBUF) & 1);
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
      // ---- sum over the slots: lane l adds the 16-byte groups l and l + 32 of every slot ---------------------------
      {
        const float4* r4 = (const float4*)(red + (size_t)q * M16_SLOTS * M16_SLOT_FLOATS);
        float4 s0 = r4[lane], s1 = r4[32 + lane];
#pragma unroll
        for (int w = 1; w < M16_SLOTS; ++w) {
          if ((uint32_t)w >= C) break;
          const float4 v0 = r4[w * (M16_SLOT_FLOATS / 4) + lane], v1 = r4[w * (M16_SLOT_FLOATS / 4) + 32 + lane];
          s0.x += v0.x; s0.y += v0.y; s0.z += v0.z; s0.w += v0.w;
          s1.x += v1.x; s1.y += v1.y; s1.z += v1.z; s1.w += v1.w;
        }
        ((float4*)tot)[lane] = s0;
        ((float4*)tot)[32 + lane] = s1;
        __syncwarp();
      }
      // ---- the 16 steps as two groups of 8 (samples A = 0..7, B = 8..15). Within a group every lane runs the steps
      // redundantly on registers (28 Gram entries, no shuffle in the dependent chain); between the groups lane l forms
      // the bracket of sample 8 + (l & 7) from its own row of the 8 x 8 cross block and the eight results are
      // gathered with shuffles. t_n = sc_n (p_n - sum_m beta_m G_nm) is the argument of the loss derivative,
      // beta_n = cf_n * f(t_n); r_n holds the bracket. --------------------------------------------------------------
      float r[B], cf[B], yv[B], sc[B], beta[B];
#pragma unroll
      for (int m = 0; m < B; ++m) {
        yv[m] = __shfl_sync(0xffffffffu, y_cur, m);
        if (LOSS == LOSS_LOGISTIC) {  // g = -y / (1 + 2^t), t = y a^n log2(e) (...)
          sc[m] = yv[m] * apw[m] * 1.4426950408889634f;
          cf[m] = -yv[m] * cfac[m];
        } else if (LOSS == LOSS_HINGE) {  // g = -y if t < 1, t = y a^n (...)
          sc[m] = yv[m] * apw[m];
          cf[m] = -yv[m] * cfac[m];
        } else {  // squared: g = t - y, t = a^n (...)
          sc[m] = apw[m];
          cf[m] = cfac[m];
        }
        if (m >= nv) cf[m] = 0.0f;  // samples beyond the chain's end take no step
      }
      float Gaa[BLK_PAIRS], Gbb[BLK_PAIRS], gba[8];
#pragma unroll
      for (int n2 = 1; n2 < 8; ++n2) {
        const float4 lo = *(const float4*)&tot[n2 * 8], hi = *(const float4*)&tot[n2 * 8 + 4];
        const float row[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
#pragma unroll
        for (int k = 0; k < 8; ++k)
          if (k < n2) Gaa[n2 * (n2 - 1) / 2 + k] = row[k];
        const float4 lo2 = *(const float4*)&tot[128 + n2 * 8], hi2 = *(const float4*)&tot[128 + n2 * 8 + 4];
        const float row2[8] = {lo2.x, lo2.y, lo2.z, lo2.w, hi2.x, hi2.y, hi2.z, hi2.w};
#pragma unroll
        for (int k = 0; k < 8; ++k)
          if (k < n2) Gbb[n2 * (n2 - 1) / 2 + k] = row2[k];
      }
      {
        const int own = 8 + (lane & 7);  // this lane's sample of group B
        const float4 lo = *(const float4*)&tot[own * 8], hi = *(const float4*)&tot[own * 8 + 4];
        gba[0] = lo.x; gba[1] = lo.y; gba[2] = lo.z; gba[3] = lo.w; gba[4] = hi.x; gba[5] = hi.y; gba[6] = hi.z; gba[7] = hi.w;
      }
#pragma unroll
      for (int m = 0; m < 8; ++m) {
        const float4 pp = *(const float4*)&tot[192 + 4 * m];  // w_hi . x, w_mid . x, w_lo . x; small terms first
        r[m] = (pp.z + pp.y) + pp.x;
      }
      float r_own;
      {
        const float4 pp = *(const float4*)&tot[192 + 4 * (8 + (lane & 7))];
        r_own = (pp.z + pp.y) + pp.x;
      }
      float p_own_a = 0.0f;  // margin of sample lane & 7 (the logistic expansion of group A is formed one sample per lane)
      if (LOSS == LOSS_LOGISTIC) {
        const float4 pp = *(const float4*)&tot[192 + 4 * (lane & 7)];
        p_own_a = (pp.z + pp.y) + pp.x;
      }
      __syncwarp();  // tot is read; the next block may overwrite it
      float mine = dl_nv;  // lane 16 publishes 1 - a^nv
      if (LOSS == LOSS_LOGISTIC) {
        // The same two groups through the 8-sample recurrence with the logistic factor expanded around each group's
        // margins (see block8_recurrence): arguments and Gram entries scaled by sc_n beforehand.
        const float sc_own = y_cur * apw_own * 1.4426950408889634f;  // of sample lane & 15
        const float sc_own_a = __shfl_sync(0xffffffffu, sc_own, lane & 7), sc_own_b = __shfl_sync(0xffffffffu, sc_own, 8 + (lane & 7));
        float t8[8], cf8[8], yv8[8], b8[8];
#pragma unroll
        for (int m = 0; m < 8; ++m) {
          t8[m] = sc[m] * r[m]; cf8[m] = cf[m]; yv8[m] = yv[m];
#pragma unroll
          for (int k2 = 0; k2 < m; ++k2) Gaa[m * (m - 1) / 2 + k2] *= sc[m];
        }
        block8_recurrence<LOSS>(t8, Gaa, cf8, yv8, sc_own_a * p_own_a, jets, b8);
#pragma unroll
        for (int m = 0; m < 8; ++m) {
          beta[m] = b8[m];
          r_own = fmaf(-b8[m], gba[m], r_own);
        }
        __syncwarp();  // every lane has read the expansions of group A
#pragma unroll
        for (int m = 0; m < 8; ++m) {
          t8[m] = sc[8 + m] * __shfl_sync(0xffffffffu, r_own, m); cf8[m] = cf[8 + m]; yv8[m] = yv[8 + m];
#pragma unroll
          for (int k2 = 0; k2 < m; ++k2) Gbb[m * (m - 1) / 2 + k2] *= sc[8 + m];
        }
        block8_recurrence<LOSS>(t8, Gbb, cf8, yv8, sc_own_b * r_own, jets, b8);
#pragma unroll
        for (int m = 0; m < 8; ++m) beta[8 + m] = b8[m];
      } else {
#pragma unroll
      for (int m = 0; m < 8; ++m) {  // group A
        const float tm_ = sc[m] * r[m];
        if (LOSS == LOSS_HINGE) beta[m] = (tm_ < 1.0f) ? cf[m] : 0.0f;
        else beta[m] = cf[m] * (tm_ - yv[m]);
#pragma unroll
        for (int n2 = m + 1; n2 < 8; ++n2) r[n2] = fmaf(-beta[m], Gaa[n2 * (n2 - 1) / 2 + m], r[n2]);
        r_own = fmaf(-beta[m], gba[m], r_own);  // off the dependent chain
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) r[8 + i] = __shfl_sync(0xffffffffu, r_own, i);
#pragma unroll
      for (int m = 0; m < 8; ++m) {  // group B
        const float tm_ = sc[8 + m] * r[8 + m];
        if (LOSS == LOSS_HINGE) beta[8 + m] = (tm_ < 1.0f) ? cf[8 + m] : 0.0f;
        else beta[8 + m] = cf[8 + m] * (tm_ - yv[8 + m]);
#pragma unroll
        for (int n2 = m + 1; n2 < 8; ++n2) r[8 + n2] = fmaf(-beta[8 + m], Gbb[n2 * (n2 - 1) / 2 + m], r[8 + n2]);
      }
      }
#pragma unroll
      for (int m = 0; m < B; ++m)
        if (lane == m) mine = beta[m] * a_nv;  // gamma_m = eta g_m a^{nv-1-m} = beta_m a^{nv}
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
    // Lane m < 16 requests this CTA's column slice of row m of a block as one bulk copy; the sixteen copies complete
    // on the stage's barrier. A stage is refilled as soon as every math warp of this CTA has run its tensor-core passes
    // over it and holds its own columns of the rows in registers (they arrive on a named barrier that this warp waits
    // on): well before the block's gamma is known, so the rows of block b + 2 have a whole block time to arrive.
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
      if (F32) {  // fp32 rows: the update of block b reads its stage, after gamma_b
        __syncthreads();
        if (gam[B + 1] != 0.0f) { stop = true; break; }
      }
      asm volatile("bar.sync 2, %0;" ::"r"(consumed_threads) : "memory");  // the stage of block b has been read
      request(requested, st);
      ++requested;
      peek(requested);
      st = (st + 1 == S) ? 0 : st + 1;
      if (!F32) {
        __syncthreads();
        if (gam[B + 1] != 0.0f) { stop = true; ++b; break; }
      }
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
  if constexpr (F32) {
    // ---- fp32 rows: Gram block and margins on the fp32 pipes ------------------------------------------------------
    // The CTA's slice is narrow here (at most 64 chunks of 4 columns: the planner spreads a chain over as many CTAs as
    // there are idle SMs), and the math threads share it as a 16 x 16 grid: thread (i, g) holds row i's chunks g,
    // g + 16, .. in registers and forms row i of the Gram block over those columns against the 16 staged rows (whose
    // chunks every thread of the same g reads at the same address). Lanes l and l ^ 16 hold the same row; their sums
    // meet with a shuffle, lanes 0..15 fill the warp's table, and the two-level sum of the tensor-core form takes over.
    // The Gram part does not depend on the model and is formed (and sent) one block ahead, while the recurrence warp
    // works; between two model updates lie the update itself (one column per thread, model in shared memory), the
    // margins from the row registers and their way through the cluster.
    // (Measured on k = 16, d = 1024, eight CTAs per chain: 2.15 ms against 2.67 ms for the 8-sample kernel with one CTA
    // per chain. The Gram block as 4 x 4 tiles over 16 column slices with a transposing sum, and the margins by 64
    // threads with one 4-byte store each, halve the shared-memory loads and measured 2.49 ms.)
    constexpr int NQ = 4;  // chunks per thread at most (checked on the host: chunks per CTA <= NQ * 16)
    const int mt = (int)threadIdx.x - 64;
    const int i16 = mt & 15, g = mt >> 4, G16 = math_threads >> 4;
    const int ncols = my_chunks * 4;
    float* wsm = (float*)w3;  // this CTA's slice of the model
    {
      const long long c0 = chunk0 * 4;
      const float* src = p.resume ? (p.W + (size_t)j * d + c0) : (p.w0 ? p.w0 + c0 : nullptr);
      for (int c = mt; c < ncols; c += math_threads) wsm[c] = src ? src[c] : 0.0f;
    }
    const uint32_t own_base = (uint32_t)__cvta_generic_to_shared(smem);
    uint32_t peer_base[8];
#pragma unroll
    for (int rr = 0; rr < 8; ++rr) peer_base[rr] = map_shared_rank(smem, (uint32_t)rr < C ? (uint32_t)rr : rank);
    asm volatile("bar.sync 4, %0;" ::"r"(math_threads) : "memory");  // the model slice is in shared memory
    cluster_barrier();  // start-up
    auto wait_rows = [&](int stg, uint32_t parity) __attribute__((always_inline)) {
      if (my_chunks > 0 && !mbar_wait_bounded(&bars[stg], parity, bp.spin_limit)) {
        set_status(p.status, DEV_TIMEOUT, 1, (long long)blockIdx.x);
        for (uint32_t rr = 0; rr < C; ++rr) st_shared_cluster(map_shared_rank((const void*)give_up, rr), 1);
      }
    };
    // adds the math warps' tables up over the 16-byte groups [g0, g0 + n) in warp order and sends the sums to this
    // CTA's slot in every CTA of the cluster (after a barrier among the math warps: the tables are written)
    auto reduce_and_send = [&](int g0, int n, int q) __attribute__((always_inline)) {
      asm volatile("bar.sync 3, %0;" ::"r"(math_threads) : "memory");
      const uint32_t ob = (uint32_t)__cvta_generic_to_shared(&pbar[q]) - own_base;
      for (int e = g0 + mt; e < g0 + n; e += math_threads) {
        const float4* p4 = (const float4*)part + e;
        float4 sum = p4[0];
#pragma unroll
        for (int w = 1; w < M16_WARPS; ++w)
          if (w < math_warps) {
            const float4 v = p4[w * (M16_SLOT_FLOATS / 4)];
            sum.x += v.x; sum.y += v.y; sum.z += v.z; sum.w += v.w;
          }
        const uint32_t od = (uint32_t)__cvta_generic_to_shared(red + ((size_t)q * M16_SLOTS + rank) * M16_SLOT_FLOATS + 4 * e) - own_base;
#pragma unroll
        for (int rr = 0; rr < 8; ++rr)
          if ((uint32_t)rr < C) st_async_f32x4(peer_base[rr] + od, sum, peer_base[rr] + ob);
      }
    };
    float4 xo[NQ];  // this thread's chunks of row i16 of the block whose margins come next
    float* tbl = part + (size_t)(warp - 2) * M16_SLOT_FLOATS;
    auto gram_part = [&](const unsigned char* stage, int q) __attribute__((always_inline)) {
      float acc[B];
#pragma unroll
      for (int k2 = 0; k2 < B; ++k2) acc[k2] = 0.0f;
#pragma unroll
      for (int it = 0; it < NQ; ++it) {
        const int qi = g + G16 * it;
        if (qi < my_chunks) {
          xo[it] = *(const float4*)(stage + (size_t)i16 * row_stride + (size_t)qi * 16);
#pragma unroll
          for (int k2 = 0; k2 < B; ++k2) {
            const float4 xk = *(const float4*)(stage + (size_t)k2 * row_stride + (size_t)qi * 16);
            acc[k2] = fmaf(xo[it].x, xk.x, fmaf(xo[it].y, xk.y, fmaf(xo[it].z, xk.z, fmaf(xo[it].w, xk.w, acc[k2]))));
          }
        } else {
          xo[it] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        }
      }
#pragma unroll
      for (int k2 = 0; k2 < B; ++k2) acc[k2] += __shfl_xor_sync(0xffffffffu, acc[k2], 16);
      if (lane < 16) {  // D0 row i16 = G[i16][0..7]; rows 8..15 also D1 row i16 - 8 = G[i16][8..15]
        *(float4*)(tbl + i16 * 8) = make_float4(acc[0], acc[1], acc[2], acc[3]);
        *(float4*)(tbl + i16 * 8 + 4) = make_float4(acc[4], acc[5], acc[6], acc[7]);
        if (i16 >= 8) {
          *(float4*)(tbl + 128 + (i16 - 8) * 8) = make_float4(acc[8], acc[9], acc[10], acc[11]);
          *(float4*)(tbl + 128 + (i16 - 8) * 8 + 4) = make_float4(acc[12], acc[13], acc[14], acc[15]);
        }
      }
      reduce_and_send(0, 48, q);
    };
    auto margin_part = [&](int q) __attribute__((always_inline)) {
      float pa = 0.0f;
#pragma unroll
      for (int it = 0; it < NQ; ++it) {
        const int qi = g + G16 * it;
        if (qi < my_chunks) {
          const float4 w4 = *(const float4*)(wsm + 4 * qi);
          pa = fmaf(xo[it].x, w4.x, fmaf(xo[it].y, w4.y, fmaf(xo[it].z, w4.z, fmaf(xo[it].w, w4.w, pa))));
        }
      }
      pa += __shfl_xor_sync(0xffffffffu, pa, 16);
      if (lane < 16) *(float4*)(tbl + 192 + 4 * i16) = make_float4(pa, 0.0f, 0.0f, 0.0f);  // one part (the bf16 form has three)
      reduce_and_send(48, 16, q);
    };
    int sg = 0, su = 0;  // stage of the next block whose Gram part is formed / whose update is applied
    uint32_t pg = 0u;
    auto gram_next = [&](long long blk) __attribute__((always_inline)) {
      wait_rows(sg, pg);
      gram_part(ring + (size_t)sg * B * row_stride, (int)(blk % NBUF));
      if (++sg == S) { sg = 0; pg ^= 1u; }
    };
    if (nb > 0) {
      gram_next(0);
      margin_part(0);
    }
    for (long long b = 0; b < nb; ++b) {
      if (b + 1 < nb) gram_next(b + 1);  // while the recurrence warp works on block b
      __syncthreads();                   // gamma_b and the decision are in gam
      if (gam[B + 1] != 0.0f) {
        // giving up: sums sent just now may still be on their way to a peer; let them land before anyone exits
        const long long t0 = clock64();
        while (clock64() - t0 < 100000) {}
        break;
      }
      // ---- w <- w - (1 - a^nv) w - sum_m gamma_m x_m, one column per thread -----------------------------------------
      {
        const float* xs = (const float*)(ring + (size_t)su * B * row_stride);
        const size_t rs4 = row_stride / 4;
        const float ndl = -gam[B];
        for (int c = mt; c < ncols; c += math_threads) {
          float wv = wsm[c];
          wv = fmaf(ndl, wv, wv);
#pragma unroll
          for (int m = 0; m < B; ++m) wv = fmaf(-gam[m], xs[(size_t)m * rs4 + c], wv);
          wsm[c] = wv;
        }
      }
      asm volatile("bar.arrive 2, %0;" ::"r"(consumed_threads) : "memory");  // this warp is done with the stage of block b
      if (++su == S) su = 0;
      asm volatile("bar.sync 4, %0;" ::"r"(math_threads) : "memory");        // the model slice is up to date
      if (b + 1 < nb) margin_part((int)((b + 1) % NBUF));
    }
    cluster_barrier();
    {
      float* dst = p.W + (size_t)j * d + chunk0 * 4;
      for (int c = mt; c < ncols; c += math_threads) dst[c] = wsm[c];
    }
  } else {
  const int mw = warp - 2;
  const int lc = mw * 32 + lane;  // this thread's 16-byte chunk within the CTA's slice
  const bool act = lc < my_chunks;
  const int warp_chunks = my_chunks - mw * 32 < 0 ? 0 : (my_chunks - mw * 32 > 32 ? 32 : my_chunks - mw * 32);
  const int ksteps = (warp_chunks + 1) / 2;  // 16 columns (two chunks) per tensor-core step
  float2 w2[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) w2[i] = make_float2(0.0f, 0.0f);
  if (act) {
    const long long c0 = chunk0 * 8 + (long long)lc * 8;
    const float* src = p.resume ? (p.W + (size_t)j * d + c0) : (p.w0 ? p.w0 + c0 : nullptr);
    if (src) {
#pragma unroll
      for (int i = 0; i < 4; ++i) w2[i] = make_float2(src[2 * i], src[2 * i + 1]);
    }
  }
  // the thread's model values as three bf16 rows: w = hi + mid + lo (each remainder is exact in fp32)
  auto publish_model = [&]() __attribute__((always_inline)) {
    if (act) {
      uint32_t hi[4], mid[4], lo[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        hi[i] = pack_bf16x2(w2[i].x, w2[i].y);
        const float rx = w2[i].x - __uint_as_float(hi[i] << 16), ry = w2[i].y - __uint_as_float(hi[i] & 0xffff0000u);
        mid[i] = pack_bf16x2(rx, ry);
        const float sx = rx - __uint_as_float(mid[i] << 16), sy = ry - __uint_as_float(mid[i] & 0xffff0000u);
        lo[i] = pack_bf16x2(sx, sy);
      }
      *(uint4*)(w3 + 0 * row_stride + (size_t)lc * 16) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
      *(uint4*)(w3 + 1 * row_stride + (size_t)lc * 16) = make_uint4(mid[0], mid[1], mid[2], mid[3]);
      *(uint4*)(w3 + 2 * row_stride + (size_t)lc * 16) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
    }
    __syncwarp();
  };
  publish_model();
  // operand tile addresses. Rows: lanes 0..7 rows 0..7 columns +0, lanes 8..15 rows 8..15 columns +0, lanes 16..23 rows
  // 0..7 columns +8, lanes 24..31 rows 8..15 columns +8: the four registers come out in the A-fragment order (a0..a3).
  // Model rows: lanes 0..7 rows (hi, mid, lo, zero x 5) columns +0, lanes 8..15 the same rows columns +8.
  const size_t warp_col_bytes = (size_t)mw * 512;
  const size_t x_off = (size_t)((lane & 7) + 8 * ((lane >> 3) & 1)) * row_stride + warp_col_bytes + (size_t)(lane >> 4) * 16;
  const unsigned char* w_src = w3 + (size_t)((lane & 7) < 3 ? (lane & 7) : 3) * row_stride + warp_col_bytes + (size_t)((lane >> 3) & 1) * 16;
  // shared-memory window of every CTA of the cluster (the same offsets apply inside each window)
  const uint32_t own_base = (uint32_t)__cvta_generic_to_shared(smem);
  uint32_t peer_base[8];
#pragma unroll
  for (int rr = 0; rr < 8; ++rr) peer_base[rr] = map_shared_rank(smem, (uint32_t)rr < C ? (uint32_t)rr : rank);
  cluster_barrier();  // start-up

  const int g8 = lane >> 2, t4 = lane & 3;
  // wait (bounded) for the rows of a block; a wait that runs out is flagged in every CTA of the cluster
  auto wait_rows = [&](int stg, uint32_t parity) __attribute__((always_inline)) {
    if (my_chunks > 0 && !mbar_wait_bounded(&bars[stg], parity, bp.spin_limit)) {
      set_status(p.status, DEV_TIMEOUT, 1, (long long)blockIdx.x);
      for (uint32_t rr = 0; rr < C; ++rr) st_shared_cluster(map_shared_rank((const void*)give_up, rr), 1);
    }
  };
  // D0, D1, D2 of a block over this warp's columns, sent to this warp's slot of every CTA of the cluster
  auto tensor_pass = [&](const unsigned char* stage, int q, uint4 (&raw)[B]) __attribute__((always_inline)) {
    float d0[2][4], d1[2][4], d2[2][4];  // two independent accumulator sets (a dependent mma takes about 20 cycles)
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
      for (int e = 0; e < 4; ++e) d0[a][e] = d1[a][e] = d2[a][e] = 0.0f;
    const unsigned char* xs = stage + x_off;
#pragma unroll
    for (int round = 0; round < 8; ++round) {
      uint32_t xa[2][4], wb[2][2];
#pragma unroll
      for (int a = 0; a < 2; ++a)
        if (round * 2 + a < ksteps) {
          ldmatrix_x4(xa[a], xs + (size_t)(round * 2 + a) * 32);
          ldmatrix_x2(wb[a], w_src + (size_t)(round * 2 + a) * 32);
        }
      // this thread's columns of two of the 16 rows, for the update: between the tensor-core steps these loads find the
      // shared-memory pipe idle; after the pass they would queue ahead of the sums that the recurrence warp waits for
#pragma unroll
      for (int a = 0; a < 2; ++a) {
        const int m = round * 2 + a;
        raw[m] = act ? *(const uint4*)(stage + (size_t)m * row_stride + (size_t)lc * 16) : make_uint4(0u, 0u, 0u, 0u);
      }
#pragma unroll
      for (int a = 0; a < 2; ++a)
        if (round * 2 + a < ksteps) {
          mma_bf16_m16n8k16(d0[a], xa[a][0], xa[a][1], xa[a][2], xa[a][3], xa[a][0], xa[a][2]);
          mma_bf16_m16n8k16(d1[a], xa[a][0], xa[a][1], xa[a][2], xa[a][3], xa[a][1], xa[a][3]);
          mma_bf16_m16n8k16(d2[a], xa[a][0], xa[a][1], xa[a][2], xa[a][3], wb[a][0], wb[a][1]);
        }
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      d0[0][e] += d0[1][e];
      d1[0][e] += d1[1][e];
      d2[0][e] += d2[1][e];
    }
    asm volatile("bar.arrive 2, %0;" ::"r"(consumed_threads) : "memory");  // this warp is done with the stage of the block
    // Two-level sum. Each warp puts its accumulators (row g8 / g8 + 8, columns 2 t4, 2 t4 + 1) into its own table of
    // this CTA; after a barrier among the math warps the first 64 math threads add the tables up in a fixed order,
    // 16 bytes each, and send the CTA's sums to this CTA's slot in every CTA of the cluster.
    float* sl = part + (size_t)mw * M16_SLOT_FLOATS;
    *(float2*)(sl + g8 * 8 + 2 * t4) = make_float2(d0[0][0], d0[0][1]);
    *(float2*)(sl + (g8 + 8) * 8 + 2 * t4) = make_float2(d0[0][2], d0[0][3]);
    *(float2*)(sl + 128 + g8 * 8 + 2 * t4) = make_float2(d1[0][2], d1[0][3]);
    if (t4 < 2) {  // columns 0..3 of D2: the three parts of p and the zero row
      *(float2*)(sl + 192 + g8 * 4 + 2 * t4) = make_float2(d2[0][0], d2[0][1]);
      *(float2*)(sl + 192 + (g8 + 8) * 4 + 2 * t4) = make_float2(d2[0][2], d2[0][3]);
    }
    asm volatile("bar.sync 3, %0;" ::"r"(math_warps * 32) : "memory");
    const uint32_t ob = (uint32_t)__cvta_generic_to_shared(&pbar[q]) - own_base;
    for (int e = mw * 32 + lane; e < M16_SLOT_FLOATS / 4; e += math_warps * 32) {
      const float4* p4 = (const float4*)part + e;
      float4 sum = p4[0];
#pragma unroll
      for (int w = 1; w < M16_WARPS; ++w)
        if (w < math_warps) {
          const float4 v = p4[w * (M16_SLOT_FLOATS / 4)];
          sum.x += v.x; sum.y += v.y; sum.z += v.z; sum.w += v.w;
        }
      const uint32_t od = (uint32_t)__cvta_generic_to_shared(red + ((size_t)q * M16_SLOTS + rank) * M16_SLOT_FLOATS + 4 * e) - own_base;
#pragma unroll
      for (int rr = 0; rr < 8; ++rr)
        if ((uint32_t)rr < C) st_async_f32x4(peer_base[rr] + od, sum, peer_base[rr] + ob);
    }
  };

  int st = 0;
  uint32_t par = 0u;
  for (long long b = 0; b < nb; ++b) {
    wait_rows(st, par);
    const unsigned char* stage = ring + (size_t)st * B * row_stride;
    uint4 raw[B];  // this thread's columns of the 16 rows, for the update
    tensor_pass(stage, (int)(b & 1), raw);
    __syncthreads();  // gamma_b and the decision are in gam; every math warp is done with the stage of block b
    if (gam[B + 1] != 0.0f) break;
    // ---- w <- w - (1 - a^nv) w - sum_m gamma_m x_m, then the model rows again -----------------------------------------
    if (act) {
      const float ndl = -gam[B];
      const float2 ndl2 = make_float2(ndl, ndl);
      float2 wv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) wv[i] = __ffma2_rn(ndl2, w2[i], w2[i]);
#pragma unroll
      for (int m = 0; m < B; ++m) {
        const float gm = -gam[m];
        const float2 g2 = make_float2(gm, gm);
        const uint32_t rw[4] = {raw[m].x, raw[m].y, raw[m].z, raw[m].w};
#pragma unroll
        for (int i = 0; i < 4; ++i)
          wv[i] = __ffma2_rn(g2, make_float2(__uint_as_float(rw[i] << 16), __uint_as_float(rw[i] & 0xffff0000u)), wv[i]);
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) w2[i] = wv[i];
    }
    publish_model();
    if (++st == S) { st = 0; par ^= 1u; }
  }
  cluster_barrier();

  if (act) {
    const long long c0 = chunk0 * 8 + (long long)lc * 8;
    float* dst = p.W + (size_t)j * d + c0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      dst[2 * i] = w2[i].x;
      dst[2 * i + 1] = w2[i].y;
    }
  }
  }  // bf16 rows
}

}  // namespace wpsgd
