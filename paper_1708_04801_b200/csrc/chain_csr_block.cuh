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
// known in advance. Here the helper warps take the next up to 64 steps (at most CSRB_EMAX nonzeros in all), give
// every distinct column among them a slot in a shared-memory hash table (linear probing, one compare-and-swap per
// nonzero), and store per nonzero its slot and value. At the block boundary all threads write the previous block's
// slots back to u and read this block's columns of u into the slots (one round trip to global memory per block, all
// loads independent); the chain warp then runs the block's steps entirely in shared memory: slot loads, a warp
// reduction, the loss derivative, slot stores. Preparation of block b + 1 (row extents, scale factors in fp64, nonzeros
// copied with cp.async, hash inserts) overlaps the steps of block b; the tables are double buffered.
//
// A row with more than CSRB_EMAX nonzeros forms a block of its own that the chain warp runs on global memory
// directly. When the scale has fallen below 1e-12 at the start of a block it is folded into u (u <- s u, s <- 1) by
// all threads; a block also ends early before the scale would leave the fp32 range of the per-step factors.
//
// Column indices are checked against d when they are inserted (a bad index sets the status word and the entry is
// dropped); the kernel has no unbounded wait: every barrier is reached by all threads the same number of times.
#pragma once

#include "chain_block.cuh"
#include "chain_csr.cuh"

namespace wpsgd {

constexpr int CSRB_STEPS = 64;          // most steps per block
constexpr int CSRB_EMAX = 4096;         // most nonzeros per block
constexpr int CSRB_HASH = 8192;         // slots of the column table (power of two, > CSRB_EMAX)
constexpr int CSRB_HASH_BITS = 13;
constexpr int CSRB_THREADS = 128;       // warp 0: chain; warps 1..3: preparation
constexpr int CSRB_HELPERS = CSRB_THREADS - 32;

struct CsrBlockMeta {
  int nsteps;    // steps in the block (0: the chain has ended)
  int nent;      // nonzeros of those steps
  int direct;    // 1: a single long row, run on global memory
  int nuniq;     // distinct columns (filled while inserting)
  float fold;    // != 0: multiply u by it before the block (the scale was folded back)
  int pad[3];
};

// One buffer of a prepared block.
struct CsrBlockBuf {
  int keys[CSRB_HASH];                 // column of every slot, -1 = free
  float val[CSRB_EMAX];                // value of every nonzero, rows one after the other
  unsigned short slot[CSRB_EMAX];      // slot of every nonzero
  unsigned short uslot[CSRB_EMAX];     // the occupied slots, in order of first insertion
  long long gbeg[CSRB_STEPS];          // first nonzero of the step's row in col_idx / val
  int rbeg[CSRB_STEPS];                // first nonzero of the step within the block
  int rcnt[CSRB_STEPS];                // nonzeros of the step's row
  float yv[CSRB_STEPS];                // label
  float sbef[CSRB_STEPS];              // scale before the step
  float eos[CSRB_STEPS];               // eta_n / scale after the step
  CsrBlockMeta meta;
};

struct CsrBlockSmem {
  CsrBlockBuf buf[2];
  float ucache[CSRB_HASH];             // u at the columns of the running block, by slot
  int colbuf[CSRB_EMAX];               // columns of the block being prepared
};

__device__ __forceinline__ void named_barrier(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

__device__ __forceinline__ int csrb_hash(int col) { return (int)(((uint32_t)col * 0x9E3779B1u) >> (32 - CSRB_HASH_BITS)); }

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
  }
  __syncthreads();

  // ---- preparation of one block (helper warps only) ------------------------------------------------------------
  long long s_next = 0;                          // first step of the next block to prepare (planner warp)
  double sc = p.resume ? p.scale[j] : 1.0;       // scale after the last planned step (planner warp)
  const double lam = (double)p.lambda, eta0 = (double)p.eta0;
  auto prepare = [&](CsrBlockBuf& B) {
    if (warp == 1) {
      float fold = 0.0f;
      if (sc < 1e-12) {
        fold = (float)sc;
        sc = 1.0;
      }
      int nsteps = 0, nent = 0, direct = 0;
      bool more = true;
      for (int part = 0; part < CSRB_STEPS / 32 && more; ++part) {
        const long long s = s_next + nsteps + lane;
        const bool valid = s < n_run;
        long long gb = 0, ge = 0;
        float yy = 0.0f;
        if (valid) {
          const uint32_t i = idx[s];
          gb = rp[i];
          ge = rp[i + 1];
          yy = yshard[i];
        }
        const long long len = ge - gb;
        const int cnt = len > (long long)CSRB_EMAX ? CSRB_EMAX + 1 : (int)len;
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
          B.gbeg[r] = gb;
          B.rbeg[r] = nent + icnt - cnt;
          B.rcnt[r] = cnt;
          B.yv[r] = yy;
          B.sbef[r] = (float)(sc * ea);
          B.eos[r] = (float)(eta / (sc * ia));
        }
        if (n_ok > 0) {
          nent += __shfl_sync(0xffffffffu, icnt, n_ok - 1);
          sc *= __shfl_sync(0xffffffffu, ia, n_ok - 1);
          nsteps += n_ok;
        }
        if (n_ok < 32) more = false;
        if (nsteps == 0 && valid && lane == 0) {
          // the first row does not fit the tables: a block of its own, run on global memory
          B.gbeg[0] = gb;
          B.rbeg[0] = 0;
          B.rcnt[0] = 0;
          B.yv[0] = yy;
          B.sbef[0] = (float)sc;
          B.eos[0] = (float)(eta / (sc * a));
        }
        const int lone = __shfl_sync(0xffffffffu, (nsteps == 0 && valid) ? 1 : 0, 0);
        if (lone) {
          direct = 1;
          nsteps = 1;
          nent = 0;
          sc *= __shfl_sync(0xffffffffu, a, 0);
          // the row length travels in gbeg[1] (unused by a block of one step)
          if (lane == 0) B.gbeg[1] = ge;
        }
      }
      if (lane == 0) {
        B.meta.nsteps = nsteps;
        B.meta.nent = nent;
        B.meta.direct = direct;
        B.meta.fold = fold;
      }
      s_next += nsteps;
    }
    named_barrier(1, CSRB_HELPERS);  // the plan of the block is in shared memory
    const int nsteps = B.meta.nsteps, nent = B.meta.nent;
    if (!B.meta.direct) {
      // nonzeros of the block's rows: asynchronous 4-byte copies, all in flight together
      for (int r = warp - 1; r < nsteps; r += CSRB_HELPERS / 32) {
        const long long g0 = B.gbeg[r];
        const int off = B.rbeg[r], cnt = B.rcnt[r];
        for (int o = lane; o < cnt; o += 32) {
          cp_async4(&sm.colbuf[off + o], p.col_idx + g0 + o);
          cp_async4(&B.val[off + o], p.val + g0 + o);
        }
      }
      cp_async_commit();
      cp_async_wait(0);
      named_barrier(1, CSRB_HELPERS);  // every helper's copies have landed
      for (int e = (int)threadIdx.x - 32; e < nent; e += CSRB_HELPERS) {
        int col = sm.colbuf[e];
        if ((unsigned long long)(long long)col >= (unsigned long long)p.d) {
          set_status(p.status, DEV_BOUNDS, 21, (long long)col);
          col = 0;
          B.val[e] = 0.0f;
        }
        int h = csrb_hash(col);
        for (int probe = 0; probe < CSRB_HASH; ++probe) {
          const int old = atomicCAS(&B.keys[h], -1, col);
          if (old == -1) {
            B.uslot[atomicAdd(&B.meta.nuniq, 1)] = (unsigned short)h;
            break;
          }
          if (old == col) break;
          h = (h + 1) & (CSRB_HASH - 1);
        }
        B.slot[e] = (unsigned short)h;
      }
    }
  };

  if (warp != 0) prepare(sm.buf[0]);
  __syncthreads();

  for (long long b = 0;; ++b) {
    CsrBlockBuf& B = sm.buf[b & 1];
    const int nsteps = B.meta.nsteps;
    if (nsteps == 0) break;
    const int nuniq = B.meta.nuniq, direct = B.meta.direct;
    const float fold = B.meta.fold;
    if (fold != 0.0f) {  // rare: the scale was folded back before this block
      for (long long c = threadIdx.x; c < p.d; c += CSRB_THREADS) u[c] = __ldcg(u + c) * fold;
      __syncthreads();
    }
    // ---- this block's columns of u into the cache (loads that bypass L1: other threads of the CTA wrote u) -------
    for (int i = threadIdx.x; i < nuniq; i += CSRB_THREADS) {
      const int h = B.uslot[i];
      sm.ucache[h] = __ldcg(u + B.keys[h]);
    }
    __syncthreads();
    if (warp != 0) {
      prepare(sm.buf[(b + 1) & 1]);
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
      const float g = loss_derivative(LOSS, B.yv[0], B.sbef[0] * acc);
      if (g != 0.0f) {
        const float coef = B.eos[0] * g;
        for (long long o = g0 + lane; o < g1; o += 32) {
          const int c = p.col_idx[o];
          if ((unsigned long long)(long long)c < (unsigned long long)p.d) u[c] = fmaf(-coef, p.val[o], __ldcg(u + c));
        }
      }
    } else {
      // ---- the block's steps, in shared memory ------------------------------------------------------------------
      constexpr int Q = 2;  // nonzeros per lane held in registers (rows of up to 64 nonzeros); longer rows loop
      int n_beg = B.rbeg[0], n_cnt = B.rcnt[0];
      float n_y = B.yv[0], n_sb = B.sbef[0], n_eos = B.eos[0];
      int n_sl[Q];
      float n_v[Q];
#pragma unroll
      for (int q = 0; q < Q; ++q) {
        const int o = lane + 32 * q;
        n_sl[q] = o < n_cnt ? B.slot[n_beg + o] : 0;
        n_v[q] = o < n_cnt ? B.val[n_beg + o] : 0.0f;
      }
      for (int r = 0; r < nsteps; ++r) {
        const int beg = n_beg, cnt = n_cnt;
        const float yy = n_y, sb = n_sb, eos = n_eos;
        int sl[Q];
        float v[Q], uq[Q];
#pragma unroll
        for (int q = 0; q < Q; ++q) {
          sl[q] = n_sl[q];
          v[q] = n_v[q];
          uq[q] = sm.ucache[sl[q]];
        }
        if (r + 1 < nsteps) {  // the next step's row does not depend on this step
          n_beg = B.rbeg[r + 1];
          n_cnt = B.rcnt[r + 1];
          n_y = B.yv[r + 1];
          n_sb = B.sbef[r + 1];
          n_eos = B.eos[r + 1];
#pragma unroll
          for (int q = 0; q < Q; ++q) {
            const int o = lane + 32 * q;
            n_sl[q] = o < n_cnt ? B.slot[n_beg + o] : 0;
            n_v[q] = o < n_cnt ? B.val[n_beg + o] : 0.0f;
          }
        }
        float acc = 0.0f;
#pragma unroll
        for (int q = 0; q < Q; ++q) acc = fmaf(uq[q], v[q], acc);
        for (int o = lane + 32 * Q; o < cnt; o += 32) acc = fmaf(sm.ucache[B.slot[beg + o]], B.val[beg + o], acc);
        acc = warp_sum(acc);
        const float g = loss_derivative(LOSS, yy, sb * acc);
        if (g != 0.0f) {
          const float coef = eos * g;
#pragma unroll
          for (int q = 0; q < Q; ++q)
            if (lane + 32 * q < cnt) sm.ucache[sl[q]] = fmaf(-coef, v[q], uq[q]);
          for (int o = lane + 32 * Q; o < cnt; o += 32) {
            const int h = B.slot[beg + o];
            sm.ucache[h] = fmaf(-coef, B.val[beg + o], sm.ucache[h]);
          }
        }
        __syncwarp();  // the next step's slot loads must see this step's stores
      }
    }
    __syncthreads();
    // ---- the block's slots back to u; its table is free again ----------------------------------------------------
    for (int i = threadIdx.x; i < nuniq; i += CSRB_THREADS) {
      const int h = B.uslot[i];
      u[B.keys[h]] = sm.ucache[h];
      B.keys[h] = -1;
    }
    if (threadIdx.x == 0) B.meta.nuniq = 0;
    __syncthreads();
  }
  if (warp == 1 && lane == 0) p.scale[j] = sc;
}

}  // namespace wpsgd
