// Blocked chains on bf16 rows with the Gram products on the 5th-generation tensor cores (tcgen05).
//
// Same blocked form of Eq. 5 as chain_block.cuh (8 samples per synchronisation), but the 8x8 Gram block
// G_mn = x_m.x_n of every block no longer costs the math warps anything: four "Gram warps" stream the rows of
// 64 consecutive samples of the chain (one super-block = 8 blocks) through shared memory, 64 columns at a
// time, in the K-major core-matrix layout that tcgen05.mma reads, and accumulate the whole 64x64 product
// X X^T in tensor memory (bf16 x bf16 products are exact, sums in fp32). Only the eight 8x8 blocks on the
// diagonal are kept. G does not depend on the model, so this runs one super-block ahead of the chain; the
// rows then reach the chain's own ring a few dozen samples later out of L2.
//
// Warps of a CTA (one CTA per node):
//   0      recurrence warp   sums p partials, 8-step recurrence, publishes gamma (as in chain_block.cuh)
//   1      copy warp         bulk copies (cp.async.bulk, never multicast) of the 8 rows of a block into the ring
//   2..5   Gram warps        16-byte asynchronous copies into core-matrix tiles, one elected thread issues
//                            tcgen05.mma, all four read the diagonal blocks back with tcgen05.ld
//   6..    math warps        model in registers; p = X_b w and the update w -= (1-a^8) w + sum gamma_m x_m
//
// Synchronisation: chain side (warps 0, 1, 6..) on two named barriers per block; Gram side on a third; the two
// sides meet through two counters in shared memory (super-blocks whose Gram blocks are published, blocks the
// chain has finished). Every wait (mbarrier, counter) is bounded; a wait that runs out ends in the status
// word, the warps of a side leave together, copies and MMAs in flight are waited for (bounded) and tensor
// memory is released before the kernel returns.
#pragma once

#include "chain_block.cuh"

namespace wpsgd {

constexpr int TC_SB = 64;        // samples per super-block (rows of one tcgen05 product)
constexpr int TC_NB = 10;        // tile buffers of the Gram stream
constexpr int TC_D = 7;          // copies run TC_D - 1 chunks ahead of the multiply; a buffer is refilled TC_NB - TC_D + 1
                                 // chunks after the multiply that read it was issued, so that wait is never on the path
constexpr int TC_TILE = 8192;    // bytes of a tile: 64 rows x 64 bf16 columns
constexpr int TC_MATH_WARPS = 8;
constexpr int TC_THREADS = 32 * (6 + TC_MATH_WARPS);
constexpr int TC_CHAIN_THREADS = 32 * (2 + TC_MATH_WARPS);  // participants of the chain-side barriers

struct TcSmem {
  size_t ring, tiles, gbuf, redP, gam, tab, bars, mma_bars, sb_bars, flags, total;
  __host__ __device__ TcSmem(int stages, size_t row_bytes) {
    ring = 0;
    tiles = (ring + (size_t)stages * BLK_B * row_bytes + 127) / 128 * 128;
    gbuf = tiles + (size_t)TC_NB * TC_TILE;                       // [2][8 blocks][8][8] floats
    redP = gbuf + 2 * 8 * 64 * sizeof(float);
    gam = redP + (size_t)TC_MATH_WARPS * BLK_B * sizeof(float);
    tab = gam + 16 * sizeof(float);
    bars = (tab + 3 * 16 * sizeof(float) + 7) / 8 * 8;            // ring stages (up to 8)
    mma_bars = bars + 8 * sizeof(unsigned long long);             // one per tile buffer
    sb_bars = mma_bars + TC_NB * sizeof(unsigned long long);      // one per accumulator (2)
    flags = sb_bars + 3 * sizeof(unsigned long long);             // (third: final drain) then the counters
    total = flags + 32;
  }
};

__device__ __forceinline__ void named_sync(int id, int count) {
  asm volatile("barrier.cta.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}
// barrier among `count` threads that also ORs a predicate over them
__device__ __forceinline__ bool named_sync_or(int id, int count, bool pred) {
  uint32_t out;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %3, 0;\n\tbarrier.cta.red.or.pred p, %1, %2, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(out)
      : "r"(id), "r"(count), "r"((uint32_t)pred)
      : "memory");
  return out != 0;
}
// Shared-memory matrix descriptor of tcgen05.mma, K-major, no swizzle: core matrices of 8 rows x 16 bytes
// (128 contiguous bytes); sbo = byte distance between 8-row groups, lbo = between the two 16-byte K halves.
__device__ __forceinline__ uint64_t umma_desc_kmajor(const void* tile, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((((uint32_t)__cvta_generic_to_shared(tile)) & 0x3FFFFu) >> 4);  // start address, bits [0,14)
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;                                // bits [16,30)
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;                                // bits [32,46)
  d |= (uint64_t)1 << 46;                                                           // descriptor version of sm_100
  return d;                                                                         // layout type 0: no swizzle
}
// Instruction descriptor, kind::f16: D = fp32, A = B = bf16, both K-major, M = 64, N = 64.
constexpr uint32_t TC_IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((64u >> 3) << 17) | ((64u >> 4) << 24);

__device__ __forceinline__ void umma_bf16_64x64x16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, bool accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
      "l"(desc_a), "l"(desc_b), "r"(TC_IDESC), "r"((uint32_t)accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(unsigned long long* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                   (uint32_t)__cvta_generic_to_shared(bar))
               : "memory");
}
// Bounded poll of a counter in shared memory until it reaches `want`; also ends when *stop becomes non-zero.
__device__ __forceinline__ bool poll_counter(volatile int* ctr, int want, volatile int* stop, long long limit) {
  for (long long i = 0; i < limit; ++i) {
    if (*ctr >= want) return true;
    if (*stop) return false;
    __nanosleep(40);
  }
  return false;
}

template <int R, int LOSS>
__global__ void __launch_bounds__(TC_THREADS, 1) chain_tc_kernel(const BlockParams bp) {
  using XT = __nv_bfloat16;
  constexpr int V = 8, QV = 2, B = BLK_B, MW = TC_MATH_WARPS, TM = 32 * MW;
  extern __shared__ __align__(128) unsigned char smem[];
  const ChainParams& p = bp.c;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int S = bp.stages;
  const int j = p.order[blockIdx.x];
  const long long n_run = p.n_steps[j];
  const long long d = p.d;
  const size_t row_bytes = (size_t)d * sizeof(XT) + 16;  // stride of a staged row in the ring
  const size_t ld_bytes = (size_t)p.ld * sizeof(XT);
  const TcSmem L(S, row_bytes);
  unsigned char* ring = smem + L.ring;
  unsigned char* tiles = smem + L.tiles;
  float* gbuf = (float*)(smem + L.gbuf);
  float* redP = (float*)(smem + L.redP);
  float* gam = (float*)(smem + L.gam);
  float* tab = (float*)(smem + L.tab);
  unsigned long long* bars = (unsigned long long*)(smem + L.bars);
  unsigned long long* mma_bars = (unsigned long long*)(smem + L.mma_bars);
  unsigned long long* sb_bars = (unsigned long long*)(smem + L.sb_bars);
  volatile int* flags = (volatile int*)(smem + L.flags);
  volatile int* give_up = flags + 0;      // chain side: a bounded wait ran out (written before barrier 1 only)
  volatile int* g_ready = flags + 1;      // super-blocks whose Gram blocks are in gbuf
  volatile int* blocks_done = flags + 2;  // blocks the chain has finished
  volatile int* g_failed = flags + 3;     // Gram side: a bounded wait ran out
  volatile int* chain_over = flags + 4;   // the chain side has left its loop
  uint32_t* tmem_holder = (uint32_t*)(flags + 5);
  const char* shard = (const char*)p.X + (size_t)p.shard_off[j] * ld_bytes;
  const float* yshard = p.y + p.shard_off[j];
  const uint32_t* idx = p.idx + p.idx_off[j];  // padded to a multiple of 64 entries, all valid rows
  const long long nb = (n_run + B - 1) / B;
  const long long nsb = (nb + 7) / 8;          // super-blocks of 8 blocks
  const int CK = (int)(d / 64);                // 64-column chunks of a row

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
    for (int s = 0; s < TC_NB; ++s) mbar_init(&mma_bars[s], 1);
    mbar_init(&sb_bars[0], 1);
    mbar_init(&sb_bars[1], 1);
    mbar_init(&sb_bars[2], 1);
    for (int i = 0; i < 5; ++i) flags[i] = 0;
    mbar_fence_init();
  }
  if (warp == 2) {  // tensor memory: two 64-column accumulators
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     (uint32_t)__cvta_generic_to_shared(tmem_holder)), "r"(128u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();  // tables, barriers, counters and the tensor-memory address are set up
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");

  if (warp == 0) {
    // =========================== recurrence warp =========================================================
    const int n = lane & (B - 1);
    float y_nxt = 0.0f;
    uint32_t id_nxt = 0u;
    if (nb > 0) y_nxt = yshard[idx[n]];
    if (nb > 1) id_nxt = idx[B + n];
    float apw[B], cfac[B];
#pragma unroll
    for (int m = 0; m < B; ++m) { apw[m] = tab[m]; cfac[m] = tab[16 + m]; }
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
        if (LOSS == LOSS_LOGISTIC) { sc[m] = yv[m] * apw[m] * 1.4426950408889634f; cf[m] = -yv[m] * cfac[m]; }
        else if (LOSS == LOSS_HINGE) { sc[m] = yv[m] * apw[m]; cf[m] = -yv[m] * cfac[m]; }
        else { sc[m] = apw[m]; cf[m] = cfac[m]; }
        if (m >= nv) cf[m] = 0.0f;
      }
      // Gram block of this block: published by the Gram warps, one super-block at a time
      const int sb = (int)(b >> 3), bi = (int)(b & 7);
      if (*g_ready <= sb) {
        if (!poll_counter(g_ready, sb + 1, g_failed, bp.spin_limit)) {
          if (lane == 0) set_status(p.status, DEV_TIMEOUT, 2, (long long)blockIdx.x);
          *give_up = 1;
        }
      }
      __threadfence_block();
      __syncwarp();
      float Gs[BLK_PAIRS];
      {
        const float* gb = gbuf + (sb & 1) * 512 + bi * 64;
#pragma unroll
        for (int n2 = 1; n2 < B; ++n2)
#pragma unroll
          for (int m = 0; m < n2; ++m) Gs[n2 * (n2 - 1) / 2 + m] = gb[n2 * 8 + m] * sc[n2];
      }
      named_sync(1, TC_CHAIN_THREADS);  // barrier 1: p_b partials are in redP
      if (*give_up) break;               // flagged before barrier 1 only: every chain-side warp sees the same value
      float pp[MW];
#pragma unroll
      for (int w = 0; w < MW; ++w) pp[w] = redP[w * B + n];
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
      float mine = dl_nv;
#pragma unroll
      for (int m = 0; m < B; ++m)
        if (lane == m) mine = beta[m] * a_nv;
      if (lane <= B) gam[lane] = mine;
      named_sync(2, TC_CHAIN_THREADS);  // barrier 2: gamma published
      if (lane == 0) *blocks_done = (int)(b + 1);
    }
    if (lane == 0) *chain_over = 1;
    return;
  }

  if (warp == 1) {
    // =========================== copy warp: ring of 8-row blocks for p and the update ========================
    const uint32_t copy_bytes = (uint32_t)((size_t)d * sizeof(XT));
    uint32_t id_next = 0u;
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
    long long requested = 0;
    for (int s = 0; s < S; ++s) {
      peek(s);
      request(s, s);
      ++requested;
    }
    peek(requested);
    int st = 0;
    long long b = 0;
    bool stop = false;
    for (; b < nb; ++b) {
      named_sync(1, TC_CHAIN_THREADS);  // barrier 1: every math warp has block b in registers
      if (*give_up) { stop = true; break; }
      request(requested, st);           // its stage takes block b + S
      ++requested;
      peek(requested);
      named_sync(2, TC_CHAIN_THREADS);  // barrier 2
      st = (st + 1 == S) ? 0 : st + 1;
    }
    if (stop) {  // leave no copy in flight into this CTA's shared memory
      long long blk = b - 1 > 0 ? b - 1 : 0;
      for (; blk < requested && blk < nb; ++blk)
        if (blk != bp.drop_block) mbar_wait_bounded(&bars[blk % S], (uint32_t)((blk / S) & 1), bp.spin_limit);
    }
    return;
  }

  if (warp < 6) {
    // =========================== Gram warps ================================================================
    const int gt = threadIdx.x - 64;   // 0..127
    const int wq = gt >> 5;            // Gram warp number 0..3
    // Copy assignment: a warp instruction moves 8 rows x 64 contiguous bytes (lane -> row lane & 7, 16-byte chunk
    // lane >> 3 of the half), so global reads are whole sectors of 8 lines and the shared-memory writes of a
    // warp fall on 8 different 16-byte bank groups in each of 4 chunk planes (no conflicts). Over its 4 copies
    // per tile a thread covers two rows, 8 (2 wq) + rr and 8 (2 wq + 1) + rr, both halves of each.
    const int rr = lane & 7, cc = lane >> 3;
    const int q = warp & 3;            // tensor-memory subpartition this warp can read: rows 16q .. 16q+15
    const uint32_t tmem = *tmem_holder;
    const long long total = nsb * CK;  // 64-column chunks over the whole chain
    // producer position (chunk being copied) and consumer position (chunk being multiplied)
    long long gi = 0; int kci = 0; long long si = 0; long long row_sb = -1;
    const char* rowptr[2] = {nullptr, nullptr};
    bool failed = false;
    auto issue_copy = [&]() {  // copy this thread's part of chunk gi into tile buffer gi % TC_NB; one group per call
      if (gi < total) {
        if (row_sb != si) {
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const int row = 8 * (2 * wq + h) + rr;
            rowptr[h] = shard + (size_t)idx[si * TC_SB + row] * ld_bytes;
            if (cc == 0 && si + 1 < nsb) {  // ask L2 for the same row slot of the next super-block
              const char* nxt = shard + (size_t)idx[(si + 1) * TC_SB + row] * ld_bytes;
              asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(nxt), "r"((uint32_t)(d * sizeof(XT))) : "memory");
            }
          }
          row_sb = si;
        }
        unsigned char* tile = tiles + (size_t)(gi % TC_NB) * TC_TILE;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int h = i >> 1, half = i & 1;         // row group 2 wq + h, chunks 4 half + cc
          const int row = 8 * (2 * wq + h) + rr, c = 4 * half + cc;
          cp_async16(tile + c * 1024 + row * 16, rowptr[h] + (size_t)kci * 128 + c * 16);
        }
        ++gi;
        if (++kci == CK) { kci = 0; ++si; }
      }
      cp_async_commit();
    };
    for (int i = 0; i < TC_D - 1; ++i) issue_copy();
    int kc = 0; long long s = 0;
    for (long long g = 0; g < total; ++g) {
      cp_async_wait(TC_D - 2);  // this thread's part of chunk g has landed (TC_D - 1 + g groups committed)
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      // all 128 parts of the tile are in place; the same barrier carries the decision to stop
      if (named_sync_or(3, 128, failed || *chain_over != 0)) break;
      const int u = (int)(g % TC_NB);
      if (gt == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const unsigned char* tile = tiles + (size_t)u * TC_TILE;
        const uint32_t acc = tmem + (uint32_t)(64 * (s & 1));
#pragma unroll
        for (int k16 = 0; k16 < 4; ++k16) {
          const uint64_t desc = umma_desc_kmajor(tile + 2 * k16 * 1024, 1024, 128);
          umma_bf16_64x64x16(acc, desc, desc, kc > 0 || k16 > 0);
        }
        umma_commit(&mma_bars[u]);                    // the tile may be refilled once these have read it
        if (kc == CK - 1) umma_commit(&sb_bars[s & 1]);  // the super-block's product is complete
      }
      // chunk g + TC_D - 1 goes into the buffer last read by the multiply of chunk g + TC_D - 1 - TC_NB
      if (g + TC_D - 1 >= TC_NB && gi < total) {
        const long long old = g + TC_D - 1 - TC_NB;
        if (!mbar_wait_bounded(&mma_bars[old % TC_NB], (uint32_t)((old / TC_NB) & 1), bp.spin_limit)) failed = true;
      }
      issue_copy();
      if (kc == CK - 1) {
        // ---- diagonal 8x8 blocks of the finished 64x64 product -> gbuf[s & 1] ---------------------------------
        if (!mbar_wait_bounded(&sb_bars[s & 1], (uint32_t)((s >> 1) & 1), bp.spin_limit)) failed = true;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        uint32_t r[16];
        const uint32_t taddr = tmem + ((uint32_t)(32 * q) << 16) + (uint32_t)(64 * (s & 1) + 16 * q);
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
            : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
              "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
            : "r"(taddr)
            : "memory");
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        // gbuf[s & 1] still holds super-block s-2 until the chain has finished it
        if (s >= 2 && !poll_counter(blocks_done, (int)(8 * (s - 1)), chain_over, bp.spin_limit) && *chain_over == 0)
          failed = true;
        if (lane < 16) {  // lane l holds row 16q + l of the product, columns 16q .. 16q+15
          const int blk = 2 * q + (lane >> 3), rr = lane & 7, coff = (lane >> 3) * 8;
          float* dst = gbuf + (s & 1) * 512 + blk * 64 + rr * 8;
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            float v = __uint_as_float(r[0]);
#pragma unroll
            for (int k2 = 0; k2 < 16; ++k2)
              if (k2 == coff + c) v = __uint_as_float(r[k2]);
            dst[c] = v;
          }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __threadfence_block();
        if (named_sync_or(3, 128, failed)) break;
        if (gt == 0) *g_ready = (int)(s + 1);
      }
      if (++kc == CK) { kc = 0; ++s; }
    }
    // nothing of this side may still be in flight when the CTA ends: own copies, then every MMA issued (one more
    // commit arrives when all of them are done), then tensor memory is released by the warp that allocated it
    cp_async_wait(0);
    if (gt == 0) {
      umma_commit(&sb_bars[2]);
      if (!mbar_wait_bounded(&sb_bars[2], 0u, bp.spin_limit)) failed = true;
    }
    if (failed) {
      set_status(p.status, DEV_TIMEOUT, 3, (long long)blockIdx.x);
      *g_failed = 1;
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    named_sync(3, 128);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (warp == 2) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(128u) : "memory");
    return;
  }

  // ============================= math warps ================================================================
  const int tm = threadIdx.x - 192;
  const int mw = warp - 6;
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
  uint4 cur[R][B];
  int st = 0;
  uint32_t par = 0u;
  for (long long b = 0; b < nb; ++b) {
    if (!mbar_wait_bounded(&bars[st], par, bp.spin_limit)) {  // rows of block b
      set_status(p.status, DEV_TIMEOUT, 1, (long long)blockIdx.x);
      *give_up = 1;
    }
    const unsigned char* stage = ring + (size_t)st * B * row_bytes;
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
      for (int m = 0; m < B; ++m)
        cur[r][m] = act[r] ? *(const uint4*)(stage + (size_t)m * row_bytes + ((size_t)r * TM + tm) * 16)
                           : make_uint4(0u, 0u, 0u, 0u);
    // ---- p_b = X_b w ---------------------------------------------------------------------------------------
    float accp[B];
#pragma unroll
    for (int m = 0; m < B; ++m) accp[m] = 0.0f;
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
      for (int qd = 0; qd < QV; ++qd)
#pragma unroll
        for (int m = 0; m < B; ++m) {
          float x[4];
          widen_quad<XT>(cur[r][m], qd, x);
#pragma unroll
          for (int e = 0; e < 4; ++e) accp[m] = fmaf(w[r][qd * 4 + e], x[e], accp[m]);
        }
    const float ptot = warp_transpose_sum8(accp);
    if ((lane & 3) == 0) redP[mw * B + (lane >> 2)] = ptot;
    named_sync(1, TC_CHAIN_THREADS);  // barrier 1: the stage of block b is free
    if (*give_up) break;
    named_sync(2, TC_CHAIN_THREADS);  // barrier 2: gamma_b is in gam
    // ---- w <- w - (1 - a^nv) w - sum_m gamma_m x_m -------------------------------------------------------------
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
        for (int qd = 0; qd < QV; ++qd) {
          float x[4];
          widen_quad<XT>(cur[r][m], qd, x);
#pragma unroll
          for (int e = 0; e < 4; ++e) w[r][qd * 4 + e] = fmaf(-gm[m], x[e], w[r][qd * 4 + e]);
        }
    }
    if (++st == S) { st = 0; par ^= 1u; }
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
