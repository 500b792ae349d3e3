// Per-node SGD chains on CSR rows (Eq. 5), a block of steps at a time through a shared-memory cache of the
// model entries those steps touch. One CTA per node: warp 0 runs the chain, the other warps prepare blocks.
//
// As in chain_csr.cuh the model of node j is w = s * u with an fp64 scalar s (the regulariser's factor
// 1 - eta_n lambda multiplies s only), and a step is
//     z = s_{n-1} (u . x);  g = L'(y, z);  s_n = s_{n-1} (1 - eta_n lambda);  u_c <- u_c - (eta_n g / s_n) x_c
// on the row's nonzeros: the iterates of Eq. 5 in exact arithmetic, for any step-size schedule.
//
// Why blocks. In the direct kernel every step pays a round trip to the model in global memory (gather, reduce,
// scatter) on its serial path. The sample stream does not depend on the model, so the rows of the next steps are
// known in advance. The helper warps take the next up to 64 steps (at most CSRB_EMAX nonzeros in all), give every
// distinct column among them a slot in a shared-memory hash table (linear probing, one compare-and-swap per
// nonzero), store per nonzero its slot and value, and read u at the block's columns into the block's cache, all
// while the chain warp runs the previous block. The chain warp runs a block's steps entirely in shared memory: slot
// loads, a warp reduction, the loss derivative, slot stores.
//
// Block boundary. The values the helpers read for block b + 1 are stale exactly at the columns block b touches, so
// at the boundary every column of block b + 1 is looked up in block b's table and, when found, takes block b's
// cached value (shared memory to shared memory). No global-memory latency is left on the chain's path: block b's
// slots are written back to u by the helpers afterwards, before they reuse its tables for block b + 2. Tables and
// caches are double buffered.
//
// Slow boundaries (rare): a row with more than CSRB_EMAX nonzeros forms a block of its own that the chain warp runs
// on global memory; when the scale has fallen below 1e-12 at the start of a block it is folded into u (u <- s u,
// s <- 1). In both cases, and for the first block, all threads write the previous block back, apply the fold, and
// read the block's columns again from global memory. A block also ends early before the scale would leave the fp32
// range of the per-step factors.
//
// Column indices are checked against d when they are inserted (a bad index sets the status word and the entry is
// dropped). The kernel has no wait on anything but CTA barriers that every thread reaches the same number of times.
#pragma once

#include <type_traits>

#include "chain_block.cuh"
#include "chain_csr.cuh"

namespace wpsgd {

constexpr int CSRB_STEPS = 64;          // most steps per block
constexpr int CSRB_EMAX = 4096;         // most nonzeros per block
constexpr int CSRB_HASH = 8192;         // slots of the column table (power of two, > CSRB_EMAX)
constexpr int CSRB_HASH_BITS = 13;
constexpr int CSRB_THREADS = 256;       // warp 0: chain; warps 1..7: preparation
constexpr int CSRB_HELPERS = CSRB_THREADS - 32;
constexpr int CSRB_BATCH = 8;           // independent global loads a thread keeps in flight

struct CsrBlockMeta {
  int nsteps;    // steps in the block (0: the chain has ended)
  int nent;      // nonzeros of those steps
  int direct;    // 1: a single long row, run on global memory
  int nuniq;     // distinct columns (filled while inserting; 0 again once the block has been written back)
  float fold;    // != 0: multiply u by it before the block (the scale was folded back)
  int wide;      // 1: some row of the block has more than 64 nonzeros
  int pad[2];
};

// One buffer of a prepared block.
struct CsrBlockBuf {
  int keys[CSRB_HASH];                 // column of every slot, -1 = free
  float val[CSRB_EMAX];                // value of every nonzero, rows one after the other
  unsigned short slot[CSRB_EMAX];      // slot of every nonzero
  unsigned short uslot[CSRB_EMAX];     // the occupied slots, in order of first insertion
  long long gbeg[CSRB_STEPS];          // first nonzero of the step's row in col_idx / val
  int4 step[CSRB_STEPS];               // per step: first nonzero within the block, nonzeros, label bits, scale-before bits
  float eos[CSRB_STEPS];               // eta_n / scale after the step
  CsrBlockMeta meta;
};

struct CsrBlockSmem {
  CsrBlockBuf buf[2];
  float ucache[2][CSRB_HASH];          // u at the columns of a block, by slot
  int colbuf[CSRB_EMAX];               // columns of the block being prepared
};

__device__ __forceinline__ void named_barrier(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// Shared-memory accesses by 32-bit shared-window address. The block buffers are chosen at run time (b & 1), so the
// hot loops name the state space themselves instead of leaving it to address-space inference.
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ float lds_f32(uint32_t a) {
  float v;
  asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(a));
  return v;
}
__device__ __forceinline__ int lds_s32(uint32_t a) {
  int v;
  asm volatile("ld.shared.s32 %0, [%1];" : "=r"(v) : "r"(a));
  return v;
}
__device__ __forceinline__ int lds_u16(uint32_t a) {
  unsigned short v;
  asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(a));
  return (int)v;
}
__device__ __forceinline__ int4 lds_s32x4(uint32_t a) {
  int4 v;
  asm volatile("ld.shared.v4.s32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
  return v;
}
__device__ __forceinline__ void sts_f32(uint32_t a, float v) { asm volatile("st.shared.f32 [%0], %1;" ::"r"(a), "f"(v) : "memory"); }
__device__ __forceinline__ void sts_u16(uint32_t a, int v) {
  asm volatile("st.shared.u16 [%0], %1;" ::"r"(a), "h"((unsigned short)v) : "memory");
}
__device__ __forceinline__ int atoms_cas(uint32_t a, int cmp, int val) {
  int old;
  asm volatile("atom.shared.cas.b32 %0, [%1], %2, %3;" : "=r"(old) : "r"(a), "r"(cmp), "r"(val) : "memory");
  return old;
}
__device__ __forceinline__ int atoms_add(uint32_t a, int val) {
  int old;
  asm volatile("atom.shared.add.s32 %0, [%1], %2;" : "=r"(old) : "r"(a), "r"(val) : "memory");
  return old;
}

__device__ __forceinline__ int csrb_hash(int col) { return (int)(((uint32_t)col * 0x9E3779B1u) >> (32 - CSRB_HASH_BITS)); }

// cache[slot] <- u[column of slot] for the block's distinct columns i = t0, t0 + stride, ...; CSRB_BATCH loads in flight.
__device__ __forceinline__ void csrb_gather(const CsrBlockBuf& B, float* cache, const float* u, int nuniq, int t0, int stride) {
  for (int base = t0; base < nuniq; base += stride * CSRB_BATCH) {
    int h[CSRB_BATCH];
    float v[CSRB_BATCH];
#pragma unroll
    for (int g = 0; g < CSRB_BATCH; ++g) {
      const int i = base + g * stride;
      h[g] = i < nuniq ? (int)B.uslot[i] : -1;
    }
#pragma unroll
    for (int g = 0; g < CSRB_BATCH; ++g) v[g] = h[g] >= 0 ? __ldcg(u + B.keys[h[g]]) : 0.0f;
#pragma unroll
    for (int g = 0; g < CSRB_BATCH; ++g)
      if (h[g] >= 0) cache[h[g]] = v[g];
  }
}

// u[column of slot] <- cache[slot] for the block's distinct columns, and the table is emptied.
__device__ __forceinline__ void csrb_scatter(CsrBlockBuf& B, const float* cache, float* u, int nuniq, int t0, int stride) {
  for (int i = t0; i < nuniq; i += stride) {
    const int h = B.uslot[i];
    u[B.keys[h]] = cache[h];
    B.keys[h] = -1;
  }
}

template <int LOSS>
__global__ void __launch_bounds__(CSRB_THREADS, 1) chain_csr_block_kernel(const CsrParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  CsrBlockSmem& sm = *reinterpret_cast<CsrBlockSmem*>(smem_raw);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int j = p.order[blockIdx.x];
  const long long n_run = p.n_steps[j];
  const long long first = p.resume ? p.first[j] : 0;
  const long long* rp = p.row_ptr + p.shard_off[j];
  const float* yshard = p.y + p.shard_off[j];
  const uint32_t* idx = p.idx + p.idx_off[j];
  float* u = p.U + (size_t)j * p.d;

  for (int i = threadIdx.x; i < CSRB_HASH; i += CSRB_THREADS) {
    sm.buf[0].keys[i] = -1;
    sm.buf[1].keys[i] = -1;
  }
  if (threadIdx.x == 0) {
    sm.buf[0].meta.nuniq = 0;
    sm.buf[1].meta.nuniq = 0;
    sm.buf[0].meta.nsteps = 0;
    sm.buf[1].meta.nsteps = 0;
    sm.buf[0].meta.direct = 0;
    sm.buf[1].meta.direct = 0;
  }
  __syncthreads();

  // ---- preparation of one block (helper warps only) ------------------------------------------------------------
  long long s_next = 0;                          // first step of the next block to prepare (planner warp)
  double sc = p.resume ? p.scale[j] : 1.0;       // scale after the last planned step (planner warp)
  const double lam = (double)p.lambda, eta0 = (double)p.eta0;
  auto prepare = [&](CsrBlockBuf& B, float* cache) {
    if (warp == 1) {
      float fold = 0.0f;
      if (sc < 1e-12 && s_next < n_run) {  // only ahead of a block that runs: the fold is applied at its start
        fold = (float)sc;
        sc = 1.0;
      }
      // row extents and labels of the next 64 steps, all loads in flight together
      constexpr int PARTS = CSRB_STEPS / 32;
      long long gb[PARTS], ge[PARTS];
      float yy[PARTS];
      uint32_t ri[PARTS];
#pragma unroll
      for (int part = 0; part < PARTS; ++part) {
        const long long s = s_next + part * 32 + lane;
        ri[part] = s < n_run ? idx[s] : 0u;
      }
#pragma unroll
      for (int part = 0; part < PARTS; ++part) {
        const long long s = s_next + part * 32 + lane;
        gb[part] = ge[part] = 0;
        yy[part] = 0.0f;
        if (s < n_run) {
          gb[part] = rp[ri[part]];
          ge[part] = rp[ri[part] + 1];
          yy[part] = yshard[ri[part]];
        }
      }
      int nsteps = 0, nent = 0, direct = 0, wide = 0;
      bool more = true;
#pragma unroll
      for (int part = 0; part < PARTS; ++part) {
        if (!more) break;
        const long long s = s_next + part * 32 + lane;
        const bool valid = s < n_run;
        const long long len = ge[part] - gb[part];
        const int cnt = len > (long long)CSRB_EMAX ? CSRB_EMAX + 1 : (len < 0 ? 0 : (int)len);
        const double eta = p.sched == LR_INV_SQRT ? eta0 / sqrt((double)(first + s + 1)) : eta0;
        const double a = valid ? 1.0 - eta * lam : 1.0;
        int icnt = cnt;
        double ia = a;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int c2 = __shfl_up_sync(0xffffffffu, icnt, o);
          const double a2 = __shfl_up_sync(0xffffffffu, ia, o);
          if (lane >= o) {
            icnt += c2;
            ia *= a2;
          }
        }
        double ea = __shfl_up_sync(0xffffffffu, ia, 1);
        if (lane == 0) ea = 1.0;
        const bool ok = valid && (nent + icnt <= CSRB_EMAX) && (sc * ea >= 1e-30);
        const unsigned mask = __ballot_sync(0xffffffffu, ok);
        const int n_ok = (mask == 0xffffffffu) ? 32 : (__ffs((int)~mask) - 1);
        if (lane < n_ok) {
          const int r = nsteps + lane;
          B.gbeg[r] = gb[part];
          B.step[r] = make_int4(nent + icnt - cnt, cnt, __float_as_int(yy[part]), __float_as_int((float)(sc * ea)));
          B.eos[r] = (float)(eta / (sc * ia));
        }
        wide |= __any_sync(0xffffffffu, lane < n_ok && cnt > 64) ? 1 : 0;
        // a first row that does not fit the tables: a block of its own, run on global memory
        const int lone = __shfl_sync(0xffffffffu, (part == 0 && n_ok == 0 && valid) ? 1 : 0, 0);
        if (lone) {
          if (lane == 0) {
            B.gbeg[0] = gb[part];
            B.gbeg[1] = ge[part];  // the row's end travels in the unused second entry
            B.step[0] = make_int4(0, 0, __float_as_int(yy[part]), __float_as_int((float)sc));
            B.eos[0] = (float)(eta / (sc * a));
          }
          direct = 1;
          nsteps = 1;
          nent = 0;
          sc *= __shfl_sync(0xffffffffu, a, 0);
          more = false;
        } else {
          if (n_ok > 0) {
            nent += __shfl_sync(0xffffffffu, icnt, n_ok - 1);
            sc *= __shfl_sync(0xffffffffu, ia, n_ok - 1);
            nsteps += n_ok;
          }
          if (n_ok < 32) more = false;
        }
      }
      if (lane == 0) {
        B.meta.nsteps = nsteps;
        B.meta.nent = nent;
        B.meta.direct = direct;
        B.meta.fold = fold;
        B.meta.wide = wide;
      }
      s_next += nsteps;
    }
    named_barrier(1, CSRB_HELPERS);  // the plan of the block is in shared memory
    const int nsteps = B.meta.nsteps, nent = B.meta.nent;
    if (!B.meta.direct && nsteps > 0) {
      // nonzeros of the block's rows: asynchronous 4-byte copies, all in flight together
      for (int r = warp - 1; r < nsteps; r += CSRB_HELPERS / 32) {
        const long long g0 = B.gbeg[r];
        const int off = B.step[r].x, cnt = B.step[r].y;
        for (int o = lane; o < cnt; o += 32) {
          cp_async4(&sm.colbuf[off + o], p.col_idx + g0 + o);
          cp_async4(&B.val[off + o], p.val + g0 + o);
        }
      }
      cp_async_commit();
      cp_async_wait(0);
      named_barrier(1, CSRB_HELPERS);  // every helper's copies have landed
      const uint32_t keys_a = smem_addr(B.keys), slot_a = smem_addr(B.slot), uslot_a = smem_addr(B.uslot);
      const uint32_t col_a = smem_addr(sm.colbuf), nuniq_a = smem_addr(&B.meta.nuniq);
      for (int e0 = 0; e0 < nent; e0 += CSRB_HELPERS) {  // the same trip count for every lane of a warp
        const int e = e0 + (int)threadIdx.x - 32;
        bool fresh = false;
        int h = 0;
        if (e < nent) {
          int col = lds_s32(col_a + 4u * (uint32_t)e);
          if ((unsigned long long)(long long)col >= (unsigned long long)p.d) {
            set_status(p.status, DEV_BOUNDS, 21, (long long)col);
            col = 0;
            B.val[e] = 0.0f;
          }
          h = csrb_hash(col);
          for (int probe = 0; probe < CSRB_HASH; ++probe) {
            const int old = atoms_cas(keys_a + 4u * (uint32_t)h, -1, col);
            if (old == -1) {
              fresh = true;
              asm volatile("prefetch.global.L2 [%0];" ::"l"(u + col));  // the block's read of u[col] follows soon
              break;
            }
            if (old == col) break;
            h = (h + 1) & (CSRB_HASH - 1);
          }
          sts_u16(slot_a + 2u * (uint32_t)e, h);
        }
        // one counter update per warp for the columns seen for the first time
        const unsigned fm = __ballot_sync(0xffffffffu, fresh);
        if (fm) {
          int base = 0;
          if (lane == 0) base = atoms_add(nuniq_a, __popc(fm));
          base = __shfl_sync(0xffffffffu, base, 0);
          if (fresh) sts_u16(uslot_a + 2u * (uint32_t)(base + __popc(fm & ((1u << lane) - 1u))), h);
        }
      }
      named_barrier(1, CSRB_HELPERS);  // the list of distinct columns is complete
      // u at the block's columns (stale where the running block writes: see the boundary)
      csrb_gather(B, cache, u, B.meta.nuniq, (int)threadIdx.x - 32, CSRB_HELPERS);
    }
  };

  // ---- the steps of a block, chain warp, in shared memory ----------------------------------------------------------
  auto run_steps = [&](CsrBlockBuf& B, float* cache, int nsteps, auto wide_tag) {
    constexpr bool WIDE = decltype(wide_tag)::value;
    const uint32_t cache_a = smem_addr(cache), step_a = smem_addr(B.step), eos_a = smem_addr(B.eos);
    const uint32_t slot_a = smem_addr(B.slot) + 2u * (uint32_t)lane, val_a = smem_addr(B.val) + 4u * (uint32_t)lane;
    // registers of the next step: its row does not depend on the running step
    int4 n_st = lds_s32x4(step_a);
    float n_eos = lds_f32(eos_a);
    uint32_t n_c0 = cache_a, n_c1 = cache_a;  // addresses of the lane's two cached model entries
    float n_v0 = 0.0f, n_v1 = 0.0f;
    if (lane < n_st.y) {
      n_c0 = cache_a + 4u * (uint32_t)lds_u16(slot_a + 2u * (uint32_t)n_st.x);
      n_v0 = lds_f32(val_a + 4u * (uint32_t)n_st.x);
    }
    if (lane + 32 < n_st.y) {
      n_c1 = cache_a + 4u * (uint32_t)lds_u16(slot_a + 2u * (uint32_t)(n_st.x + 32));
      n_v1 = lds_f32(val_a + 4u * (uint32_t)(n_st.x + 32));
    }
    for (int r = 0; r < nsteps; ++r) {
      const int beg = n_st.x, cnt = n_st.y;
      const float yy = __int_as_float(n_st.z), sb = __int_as_float(n_st.w), eos = n_eos;
      const uint32_t c0 = n_c0, c1 = n_c1;
      const float v0 = n_v0, v1 = n_v1;
      const bool in0 = lane < cnt, in1 = lane + 32 < cnt;
      float uq0 = 0.0f, uq1 = 0.0f;
      if (in0) uq0 = lds_f32(c0);
      if (in1) uq1 = lds_f32(c1);
      if (r + 1 < nsteps) {
        n_st = lds_s32x4(step_a + 16u * (uint32_t)(r + 1));
        n_eos = lds_f32(eos_a + 4u * (uint32_t)(r + 1));
        n_v0 = n_v1 = 0.0f;
        if (lane < n_st.y) {
          n_c0 = cache_a + 4u * (uint32_t)lds_u16(slot_a + 2u * (uint32_t)n_st.x);
          n_v0 = lds_f32(val_a + 4u * (uint32_t)n_st.x);
        }
        if (lane + 32 < n_st.y) {
          n_c1 = cache_a + 4u * (uint32_t)lds_u16(slot_a + 2u * (uint32_t)(n_st.x + 32));
          n_v1 = lds_f32(val_a + 4u * (uint32_t)(n_st.x + 32));
        }
      }
      float part = fmaf(uq1, v1, uq0 * v0);
      if (WIDE)
        for (int o = lane + 64; o < cnt; o += 32) part = fmaf(cache[B.slot[beg + o]], B.val[beg + o], part);
      const float acc = warp_sum(part);  // shuffles only: nothing here waits on shared memory
      const float g = loss_derivative(LOSS, yy, sb * acc);
      const float coef = eos * g;  // g == 0 (hinge off the margin): the stores below rewrite the same values
      if (in0) sts_f32(c0, fmaf(-coef, v0, uq0));
      if (in1) sts_f32(c1, fmaf(-coef, v1, uq1));
      if (WIDE)
        for (int o = lane + 64; o < cnt; o += 32) {
          const int h = B.slot[beg + o];
          cache[h] = fmaf(-coef, B.val[beg + o], cache[h]);
        }
      __syncwarp();  // the next step's slot loads see this step's stores
    }
  };

  if (warp != 0) prepare(sm.buf[0], sm.ucache[0]);
  __syncthreads();

  int prev_direct = 0;
  for (long long b = 0;; ++b) {
    CsrBlockBuf& B = sm.buf[b & 1];
    CsrBlockBuf& Bp = sm.buf[(b + 1) & 1];  // the block that has just run (and the buffer of the next preparation)
    float* cache = sm.ucache[b & 1];
    float* cache_p = sm.ucache[(b + 1) & 1];
    const int nsteps = B.meta.nsteps, nuniq = B.meta.nuniq, direct = B.meta.direct;
    const int nuniq_p = Bp.meta.nuniq;
    const float fold = B.meta.fold;
    const bool slow = b == 0 || nsteps == 0 || fold != 0.0f || direct || prev_direct;
    if (!slow) {
      // ---- boundary: columns that the block that has just run also holds take its values -----------------------------
      const uint32_t uslot_a = smem_addr(B.uslot), keys_a = smem_addr(B.keys), keysp_a = smem_addr(Bp.keys);
      const uint32_t cache_a = smem_addr(cache), cachep_a = smem_addr(cache_p);
      for (int i = threadIdx.x; i < nuniq; i += CSRB_THREADS) {
        const int h2 = lds_u16(uslot_a + 2u * (uint32_t)i);
        const int col = lds_s32(keys_a + 4u * (uint32_t)h2);
        int h = csrb_hash(col);
        for (int probe = 0; probe < CSRB_HASH; ++probe) {
          const int k2 = lds_s32(keysp_a + 4u * (uint32_t)h);
          if (k2 == col) {
            sts_f32(cache_a + 4u * (uint32_t)h2, lds_f32(cachep_a + 4u * (uint32_t)h));
            break;
          }
          if (k2 == -1) break;
          h = (h + 1) & (CSRB_HASH - 1);
        }
      }
      __syncthreads();
    } else {
      // ---- slow boundary: write back, fold, read again ------------------------------------------------------------------
      csrb_scatter(Bp, cache_p, u, nuniq_p, threadIdx.x, CSRB_THREADS);
      __syncthreads();
      if (threadIdx.x == 0) Bp.meta.nuniq = 0;
      if (nsteps == 0) break;
      if (fold != 0.0f) {
        for (long long c = threadIdx.x; c < p.d; c += CSRB_THREADS) u[c] = __ldcg(u + c) * fold;
        __syncthreads();
      }
      csrb_gather(B, cache, u, nuniq, threadIdx.x, CSRB_THREADS);
      __syncthreads();
    }
    if (warp != 0) {
      // the block that has just run goes back to u (a slow boundary has done it already: nothing left to do), then its
      // tables and cache take the block after this one
      csrb_scatter(Bp, cache_p, u, Bp.meta.nuniq, (int)threadIdx.x - 32, CSRB_HELPERS);
      named_barrier(1, CSRB_HELPERS);
      if (threadIdx.x == 32) Bp.meta.nuniq = 0;
      named_barrier(1, CSRB_HELPERS);
      prepare(Bp, cache_p);
    } else if (direct) {
      // ---- a single long row, on global memory ---------------------------------------------------------------
      const long long g0 = B.gbeg[0], g1 = B.gbeg[1];
      float acc = 0.0f;
      for (long long o = g0 + lane; o < g1; o += 32) {
        const int c = p.col_idx[o];
        if ((unsigned long long)(long long)c < (unsigned long long)p.d) acc = fmaf(__ldcg(u + c), p.val[o], acc);
        else set_status(p.status, DEV_BOUNDS, 22, (long long)c);
      }
      acc = warp_sum(acc);
      const float g = loss_derivative(LOSS, __int_as_float(B.step[0].z), __int_as_float(B.step[0].w) * acc);
      if (g != 0.0f) {
        const float coef = B.eos[0] * g;
        for (long long o = g0 + lane; o < g1; o += 32) {
          const int c = p.col_idx[o];
          if ((unsigned long long)(long long)c < (unsigned long long)p.d) u[c] = fmaf(-coef, p.val[o], __ldcg(u + c));
        }
      }
    } else if (B.meta.wide) {
      run_steps(B, cache, nsteps, std::true_type());
    } else {
      run_steps(B, cache, nsteps, std::false_type());
    }
    prev_direct = direct;
    __syncthreads();
  }
  if (warp == 1 && lane == 0) p.scale[j] = sc;
}

}  // namespace wpsgd
