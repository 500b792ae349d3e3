// C ABI of the WP-SGD library (see include/wpsgd.h): context, host-side planning (validation,
// delays and Eq. 6 / Eq. 8 weights in fp64, node ordering, kernel selection) and kernel launches.
#include "../../include/wpsgd.h"

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <functional>
#include <numeric>
#include <string>
#include <vector>

#include "chain_block.cuh"
#include "chain_csr.cuh"
#include "chain_csr_block.cuh"
#include "chain_mma.cuh"
#include "chain_mma16.cuh"
#include "chain_dense.cuh"
#include "combine.cuh"
#include "philox.cuh"

using namespace wpsgd;

struct wpsgd_ctx {
  int device = 0;
  cudaStream_t stream = nullptr;
  int k = 0;
  long long d = 0;
  // models
  float* W = nullptr;       // [k, d]
  double* scale = nullptr;  // [k] (sparse path: w_j = scale_j * W[j])
  bool scaled = false;
  // per-launch tables on the device
  long long* t_shard_off = nullptr;  // [k+1]
  long long* t_steps = nullptr;      // [k]
  long long* t_first = nullptr;      // [k]
  long long* t_idx_off = nullptr;    // [k+1]
  long long* t_rows = nullptr;       // [k]
  long long* t_count = nullptr;      // [k] entries of the sample stream per node (steps rounded up to 8)
  int* t_order = nullptr;            // [k]
  int* t_ids = nullptr;              // [k] node numbers entering the sample stream
  int* t_group = nullptr;            // [k + 8] node of every (CTA, warp) slot of the warp-per-node blocked kernel
  double* t_weights = nullptr;       // [k]
  uint32_t* idx = nullptr;
  size_t idx_cap = 0;  // entries
  DevStatus* status = nullptr;
  double* part = nullptr;  // objective partial sums
  size_t part_cap = 0;     // doubles
  // staging of the host-buffer entry point
  void* st_X = nullptr;
  size_t st_X_cap = 0;
  float* st_y = nullptr;
  size_t st_y_cap = 0;
  float* st_v = nullptr;   // [d]
  long long* st_rp = nullptr;  // CSR staging of the host-buffer entry point
  size_t st_rp_cap = 0;
  int* st_ci = nullptr;
  size_t st_ci_cap = 0;
  float* st_va = nullptr;
  size_t st_va_cap = 0;
  float* st_w0 = nullptr;  // [d]
  // state of the chains
  bool have_run = false;
  std::vector<long long> steps_done;
  std::vector<int> node_ids;
  std::vector<long long> last_steps;  // step counts of the launch being prepared
  float eta0 = 0.f, lambda = 0.f;
  int sched = 0, loss = 0;
  uint64_t seed = 0;
  // options
  int opt_stages = 0;
  int opt_variant = 0, opt_prefetch = 0, opt_threads = 0, opt_cluster = 0;
  int opt_block_samples = 0;   // tensor-core cluster kernel: samples per block (0: chosen here, 8 or 16)
  int opt_sparse_variant = 0;  // 0: chosen here, 1: one step per round trip, 2: blocks of steps through a shared-memory cache
  long long opt_spin_limit = 1ll << 20;
  long long opt_drop_block = -1;
  int opt_sampling = 0;  // 0: i.i.d. draws, 1: one shuffle per node, cycled
  int opt_timing = 0;
  int opt_host_pipeline = 1;  // host-buffer entry point: copy the shards in groups and start chains as they arrive
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_group[4] = {nullptr, nullptr, nullptr, nullptr};
  cudaEvent_t ev0 = nullptr, ev1 = nullptr;
  bool ev_valid = false;
  long long launches = 0;
  std::string err;
};

namespace {

std::string g_err;  // last error of context-free calls

struct DeviceGuard {
  int prev = -1;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
    if (prev != dev) cudaSetDevice(dev);
    else prev = -1;
  }
  ~DeviceGuard() {
    if (prev >= 0) cudaSetDevice(prev);
  }
};

wpsgd_status fail(wpsgd_ctx* c, wpsgd_status s, const std::string& msg) {
  if (c) c->err = msg;
  else g_err = msg;
  return s;
}

#define CU_TRY(ctx, expr)                                                                          \
  do {                                                                                             \
    cudaError_t e_ = (expr);                                                                       \
    if (e_ != cudaSuccess) {                                                                       \
      const bool oom_ = (e_ == cudaErrorMemoryAllocation);                                         \
      return fail(ctx, oom_ ? WPSGD_ERR_ALLOC : WPSGD_ERR_CUDA,                                    \
                  std::string(#expr) + ": " + cudaGetErrorString(e_));                             \
    }                                                                                              \
  } while (0)

template <typename T>
wpsgd_status grow(wpsgd_ctx* c, T** p, size_t* cap, size_t need) {
  if (need <= *cap) return WPSGD_OK;
  if (*p) {
    CU_TRY(c, cudaStreamSynchronize(c->stream));
    CU_TRY(c, cudaFree(*p));
    *p = nullptr;
    *cap = 0;
  }
  const size_t want = need + need / 8;
  void* q = nullptr;
  CU_TRY(c, cudaMalloc(&q, want * sizeof(T)));
  *p = (T*)q;
  *cap = want;
  return WPSGD_OK;
}

// ---- Eq. 6 / Eq. 8 in fp64 -------------------------------------------------------------------------
// log of r^{T_j} (or of the product of skipped per-step factors for the decaying schedule)
wpsgd_status log_rates(const long long* n, int k, double eta0, int sched, double lambda, double r,
                       std::vector<double>* lg, std::string* why) {
  long long t = 0;
  for (int j = 0; j < k; ++j) {
    if (n[j] < 0) {
      *why = "negative step count";
      return WPSGD_ERR_INVALID_ARG;
    }
    t = std::max(t, n[j]);
  }
  lg->assign(k, 0.0);
  const bool given = r > 0.0;  // false for NaN
  if (given) {
    const double lr = std::log(r);
    for (int j = 0; j < k; ++j) (*lg)[j] = (double)(t - n[j]) * lr;
  } else if (sched == WPSGD_LR_CONST) {
    const double lr = std::log1p(-eta0 * lambda);
    for (int j = 0; j < k; ++j) (*lg)[j] = (double)(t - n[j]) * lr;
  } else {
    // sum_{s = n_j + 1}^{t} log(1 - eta_s lambda): suffix sums from the smallest n_j upward
    long long lo = t;
    for (int j = 0; j < k; ++j) lo = std::min(lo, n[j]);
    std::vector<double> suf((size_t)(t - lo) + 1, 0.0);  // suf[i] = sum over s in (lo + i, t]
    for (long long s = t; s > lo; --s)
      suf[(size_t)(s - 1 - lo)] = suf[(size_t)(s - lo)] + std::log1p(-eta0 / std::sqrt((double)s) * lambda);
    for (int j = 0; j < k; ++j) (*lg)[j] = suf[(size_t)(n[j] - lo)];
  }
  return WPSGD_OK;
}

wpsgd_status weights_host(const long long* n, int k, float eta0, int sched, float lambda, double r, double* w,
                          int* cond, double* sum_rT, std::string* why) {
  if (!n || !w || k < 1) {
    *why = "weights: null argument or k < 1";
    return WPSGD_ERR_INVALID_ARG;
  }
  if (sched != WPSGD_LR_CONST && sched != WPSGD_LR_INV_SQRT) {
    *why = "weights: unknown schedule";
    return WPSGD_ERR_INVALID_ARG;
  }
  std::vector<double> lg;
  wpsgd_status s = log_rates(n, k, (double)eta0, sched, (double)lambda, r, &lg, why);
  if (s != WPSGD_OK) return s;
  const double mx = *std::max_element(lg.begin(), lg.end());
  double tot = 0.0, tot_raw = 0.0;
  for (int j = 0; j < k; ++j) {
    tot += std::exp(lg[j] - mx);
    tot_raw += std::exp(lg[j]);
  }
  for (int j = 0; j < k; ++j) w[j] = std::exp(lg[j] - mx) / tot;
  if (sum_rT) *sum_rT = tot_raw;
  if (cond) *cond = (2.0 * tot_raw > std::sqrt((double)k) + (double)k) ? 1 : 0;
  return WPSGD_OK;
}

// Waits for the stream, reads a device status word and maps it; a problem found is cleared after it has been reported.
wpsgd_status read_status(wpsgd_ctx* c, DevStatus* dev_status, cudaStream_t stream) {
  DevStatus h;
  CU_TRY(c, cudaMemcpyAsync(&h, dev_status, sizeof(h), cudaMemcpyDeviceToHost, stream));
  CU_TRY(c, cudaStreamSynchronize(stream));
  if (h.code == DEV_OK) return WPSGD_OK;
  char buf[200];
  const char* what = h.code == DEV_TIMEOUT ? "a bounded device-side wait gave up" : "a device-side check of the input failed";
  snprintf(buf, sizeof(buf), "%s: device status %d at %d (detail %lld)", what, h.code, h.where, h.detail);
  cudaMemsetAsync(dev_status, 0, sizeof(DevStatus), stream);
  return fail(c, h.code == DEV_TIMEOUT ? WPSGD_ERR_TIMEOUT : WPSGD_ERR_CUDA, buf);
}

int grid_for(long long work_items, int block, int cap = 148 * 16) {
  long long g = (work_items + block - 1) / block;
  return (int)std::max(1ll, std::min<long long>(g, cap));
}

// ---- common part of run / continue: tables, sample stream ---------------------------------------------
struct Plan {
  std::vector<long long> off, steps, first, idx_off, rows, count;
  std::vector<int> order;
  long long total = 0;
};

wpsgd_status make_plan(wpsgd_ctx* c, const long long* shard_off, const long long* n_steps,
                       const std::vector<long long>& first, Plan* pl) {
  const int k = c->k;
  if (!shard_off || !n_steps) return fail(c, WPSGD_ERR_INVALID_ARG, "shard_off / n_steps is NULL");
  if (shard_off[0] < 0) return fail(c, WPSGD_ERR_INVALID_ARG, "shard_off[0] < 0");
  pl->off.assign(shard_off, shard_off + k + 1);
  pl->steps.assign(n_steps, n_steps + k);
  pl->first = first;
  pl->idx_off.assign(k + 1, 0);
  pl->rows.assign(k, 0);
  pl->count.assign(k, 0);
  for (int j = 0; j < k; ++j) {
    const long long m = shard_off[j + 1] - shard_off[j];
    if (m < 0) return fail(c, WPSGD_ERR_INVALID_ARG, "shard_off is not non-decreasing");
    if (n_steps[j] < 0) return fail(c, WPSGD_ERR_INVALID_ARG, "negative step count");
    if (n_steps[j] > 0 && m < 1) return fail(c, WPSGD_ERR_INVALID_ARG, "a node with steps has an empty shard");
    if (m > 0xFFFFFFFFll) return fail(c, WPSGD_ERR_INVALID_ARG, "a shard has 2^32 rows or more");
    pl->rows[j] = m;
    // the stream of a node is produced up to the next multiple of 64 steps (the draws simply continue), so
    // that kernels that take samples in groups of 8 or 64 always read valid rows
    pl->count[j] = (n_steps[j] + 63) / 64 * 64;
    pl->idx_off[j + 1] = pl->idx_off[j] + pl->count[j];
  }
  pl->total = pl->idx_off[k];
  pl->order.resize(k);
  std::iota(pl->order.begin(), pl->order.end(), 0);
  std::stable_sort(pl->order.begin(), pl->order.end(), [&](int a, int b) { return n_steps[a] > n_steps[b]; });
  return WPSGD_OK;
}

wpsgd_status upload_plan_and_stream(wpsgd_ctx* c, const Plan& pl) {
  const int k = c->k;
  wpsgd_status s = grow(c, &c->idx, &c->idx_cap, (size_t)std::max(1ll, pl.total));
  if (s != WPSGD_OK) return s;
  // pageable sources: the copy has left the host buffer when cudaMemcpyAsync returns
  CU_TRY(c, cudaMemcpyAsync(c->t_shard_off, pl.off.data(), (k + 1) * sizeof(long long), cudaMemcpyHostToDevice, c->stream));
  CU_TRY(c, cudaMemcpyAsync(c->t_steps, pl.steps.data(), k * sizeof(long long), cudaMemcpyHostToDevice, c->stream));
  CU_TRY(c, cudaMemcpyAsync(c->t_first, pl.first.data(), k * sizeof(long long), cudaMemcpyHostToDevice, c->stream));
  CU_TRY(c, cudaMemcpyAsync(c->t_idx_off, pl.idx_off.data(), (k + 1) * sizeof(long long), cudaMemcpyHostToDevice, c->stream));
  CU_TRY(c, cudaMemcpyAsync(c->t_rows, pl.rows.data(), k * sizeof(long long), cudaMemcpyHostToDevice, c->stream));
  CU_TRY(c, cudaMemcpyAsync(c->t_count, pl.count.data(), k * sizeof(long long), cudaMemcpyHostToDevice, c->stream));
  CU_TRY(c, cudaMemcpyAsync(c->t_order, pl.order.data(), k * sizeof(int), cudaMemcpyHostToDevice, c->stream));
  CU_TRY(c, cudaMemcpyAsync(c->t_ids, c->node_ids.data(), k * sizeof(int), cudaMemcpyHostToDevice, c->stream));
  if (pl.total > 0) {
    const long long longest = *std::max_element(pl.steps.begin(), pl.steps.end());
    dim3 grid((unsigned)grid_for(c->opt_sampling ? longest + 8 : (longest + 3) / 4 + 3, 256, 1024), (unsigned)std::min(k, 65535));
    index_stream_kernel<<<grid, 256, 0, c->stream>>>(c->opt_sampling, c->seed, k, c->t_idx_off, c->t_first, c->t_count, c->t_rows, c->t_ids, c->idx);
    CU_TRY(c, cudaGetLastError());
    c->launches++;
  }
  return WPSGD_OK;
}

wpsgd_status check_hyper(wpsgd_ctx* c, float eta0, int sched, float lambda, int loss) {
  if (!(eta0 >= 0.0f) || !std::isfinite(eta0)) return fail(c, WPSGD_ERR_INVALID_ARG, "eta0 must be finite and >= 0");
  if (!(lambda >= 0.0f) || !std::isfinite(lambda)) return fail(c, WPSGD_ERR_INVALID_ARG, "lambda must be finite and >= 0");
  if (!((double)eta0 * (double)lambda < 1.0)) return fail(c, WPSGD_ERR_INVALID_ARG, "eta * lambda must be < 1");
  if (sched != WPSGD_LR_CONST && sched != WPSGD_LR_INV_SQRT) return fail(c, WPSGD_ERR_INVALID_ARG, "unknown schedule");
  if (loss < 0 || loss > 2) return fail(c, WPSGD_ERR_INVALID_ARG, "unknown loss");
  return WPSGD_OK;
}

wpsgd_status timing_begin(wpsgd_ctx* c) {
  c->ev_valid = false;
  if (!c->opt_timing) return WPSGD_OK;
  if (!c->ev0) {
    CU_TRY(c, cudaEventCreate(&c->ev0));
    CU_TRY(c, cudaEventCreate(&c->ev1));
  }
  CU_TRY(c, cudaEventRecord(c->ev0, c->stream));
  return WPSGD_OK;
}

wpsgd_status timing_end(wpsgd_ctx* c) {
  if (!c->opt_timing) return WPSGD_OK;
  CU_TRY(c, cudaEventRecord(c->ev1, c->stream));
  c->ev_valid = true;
  return WPSGD_OK;
}

// ---- dense chain launch ---------------------------------------------------------------------------------
template <typename XT, int R, int PF>
wpsgd_status launch_reg(wpsgd_ctx* c, const ChainParams& p, bool block_per_node, int threads) {
  if (block_per_node) {
    chain_reg_kernel<XT, R, PF, true><<<p.k, threads, 0, c->stream>>>(p);
  } else {
    const int nodes_per_cta = 4;
    chain_reg_kernel<XT, R, PF, false><<<(p.k + nodes_per_cta - 1) / nodes_per_cta, 32 * nodes_per_cta, 0, c->stream>>>(p);
  }
  CU_TRY(c, cudaGetLastError());
  c->launches++;
  return WPSGD_OK;
}

template <typename XT, int R>
wpsgd_status launch_reg_pf(wpsgd_ctx* c, const ChainParams& p, bool bpn, int threads, int pf) {
  switch (pf) {
    case 2: return launch_reg<XT, R, 2>(c, p, bpn, threads);
    case 4: return launch_reg<XT, R, 4>(c, p, bpn, threads);
    default: return launch_reg<XT, R, 8>(c, p, bpn, threads);
  }
}

// ---- blocked chain kernel: shapes it takes, ring depth, launch ------------------------------------------------
constexpr size_t kSmemBudget = 220 * 1024;

template <typename XT>
bool block_kernel_fits(const wpsgd_ctx* c, bool aligned, int* threads_out, int* R_out, int* stages_out) {
  constexpr int V = XVec<XT>::V;
  if (!aligned) return false;
  if ((double)c->eta0 * (double)c->lambda > 0.25) return false;  // keeps a^-8 harmless in fp32
  const long long chunks = c->d / V;
  // up to 8 math warps with one chunk per thread (two register copies of a block: Gram products overlap the
  // recurrence); wider rows take up to 16 math warps, then two chunks per thread
  int max_threads = chunks <= 256 ? 256 : 512;
  // fp32 rows of 129..256 chunks: four math warps with two chunks per thread (one register copy, Gram and p in one pass)
  // beat eight warps with the overlapped schedule: half as many cross-lane reductions per block, and the recurrence
  // warp runs while the math warps are idle (k = 16, d = 1024: 2.67 ms against 2.84 ms)
  if (sizeof(XT) == 4 && chunks > 128 && chunks <= 256) max_threads = 128;
  if (c->opt_threads >= 64 && c->opt_threads % 32 == 0) max_threads = std::min(512, c->opt_threads);
  const int math_threads = (int)std::min<long long>(max_threads, (chunks + 31) / 32 * 32);
  int R = (int)((chunks + math_threads - 1) / math_threads);
  if (R > 2) return false;  // beyond two chunks per thread the rows of a block no longer fit in registers
  const size_t row_bytes = (size_t)c->d * sizeof(XT) + (sizeof(XT) == 2 ? 16 : 0);  // bf16 rows are staged with padding
  int stages = c->opt_stages > 0 ? c->opt_stages : 4;
  if (stages > 8) stages = 8;
  while (stages >= 2 && BlockSmem(stages, row_bytes, math_threads / 32).total > kSmemBudget) --stages;
  if (stages < 2) return false;
  *threads_out = math_threads + 64;
  *R_out = R;
  *stages_out = stages;
  return true;
}

template <typename XT, int R, bool OVL, int MAXW>
wpsgd_status launch_block_r(wpsgd_ctx* c, const BlockParams& bp, int threads, size_t smem) {
  auto go = [&](auto kern) -> wpsgd_status {
    CU_TRY(c, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    kern<<<bp.c.k, threads, smem, c->stream>>>(bp);
    CU_TRY(c, cudaGetLastError());
    c->launches++;
    return WPSGD_OK;
  };
  switch (c->loss) {
    // one 16-byte chunk per thread: room for two register copies of a block, so the Gram products of the
    // next block overlap the serial recurrence; more chunks: one copy, Gram and p in the same pass
    case WPSGD_LOSS_HINGE: return go(chain_block_kernel<XT, R, LOSS_HINGE, OVL, MAXW>);
    case WPSGD_LOSS_LOGISTIC: return go(chain_block_kernel<XT, R, LOSS_LOGISTIC, OVL, MAXW>);
    default: return go(chain_block_kernel<XT, R, LOSS_SQUARED, OVL, MAXW>);
  }
}

template <typename XT>
wpsgd_status launch_block(wpsgd_ctx* c, const ChainParams& p, int threads, int R, int stages) {
  BlockParams bp;
  bp.c = p;
  bp.stages = stages;
  bp.eta_lambda = (double)c->eta0 * (double)c->lambda;
  bp.spin_limit = c->opt_spin_limit;
  bp.drop_block = c->opt_drop_block;
  bp.group_order = nullptr;
  const size_t smem = BlockSmem(stages, (size_t)c->d * sizeof(XT) + (sizeof(XT) == 2 ? 16 : 0), threads / 32 - 2).total;
  const bool wide = threads > 64 + 32 * 8;  // more than 8 math warps: registers allow one copy of a block only
  // one register copy of a block, except fp32 rows of at most 8 math warps with one chunk per thread (two copies:
  // the Gram products of the next block overlap the recurrence)
  if (R == 1) {
    if (wide) return launch_block_r<XT, 1, false, 16>(c, bp, threads, smem);
    return sizeof(XT) == 2 ? launch_block_r<XT, 1, false, 8>(c, bp, threads, smem)
                           : launch_block_r<XT, 1, true, 8>(c, bp, threads, smem);
  }
  return wide ? launch_block_r<XT, 2, false, 16>(c, bp, threads, smem) : launch_block_r<XT, 2, false, 8>(c, bp, threads, smem);
}

// ---- bf16 rows: Gram block and margins on the tensor cores, columns split over a cluster -------------------------------
struct ClusterShape {
  int C = 1, cpc = 0, math_warps = 1, stages = 2;
  int block = 8;    // samples per block
  int stages16 = 0; // ring depth of the 16-sample form (0: it does not fit)
};

bool mma_kernel_fits(const wpsgd_ctx* c, bool aligned, ClusterShape* out) {
  if (!aligned) return false;
  if ((double)c->eta0 * (double)c->lambda > 0.25) return false;
  const long long chunks = c->d / 8;
  if (chunks < 1) return false;
  int C = c->opt_cluster;
  if (C <= 0) {
    // as few CTAs per chain as the row width allows (a CTA takes at most 8 math warps of 32 chunks): the kernel runs
    // one CTA per SM, and what a wider cluster gains in the tensor-core pass it loses in chains running at the same
    // time (measured on k = 128, d = 4096: 7.95 ms with two CTAs per chain, 9.9 ms with four, 14.0 ms with eight)
    C = 1;
    while ((chunks + C - 1) / C > 256 && C < 8) C *= 2;
  }
  if (C != 1 && C != 2 && C != 4 && C != 8) return false;
  const long long cpc = (chunks + C - 1) / C;
  if ((long long)(C - 1) * cpc >= chunks) return false;  // every CTA of the cluster owns at least one chunk
  // one 16-byte chunk of a row per lane, up to 8 math warps per CTA
  const long long mw = (cpc + 31) / 32;
  const int slots = MMA_SLOTS;
  if (mw > 8 || mw * C > slots) return false;
  // ring depth: as deep as asked for (default 2: a stage is free again as soon as its block has been through the
  // tensor-core pass, and a shallow ring lets more CTAs share an SM) while two CTAs still share an SM; else one per SM
  const size_t two_per_sm = (size_t)(227 * 1024) / 2 - 1024;
  int want = c->opt_stages > 0 ? std::min(c->opt_stages, 8) : 2;
  int stages = want;
  while (stages > 2 && MmaSmem(stages, (size_t)cpc * 16, slots).total > two_per_sm) --stages;
  if (MmaSmem(stages, (size_t)cpc * 16, slots).total > two_per_sm) {
    stages = want;
    while (stages >= 2 && MmaSmem(stages, (size_t)cpc * 16, slots).total > kSmemBudget) --stages;
    if (stages < 2) return false;
  }
  out->C = C;
  out->cpc = (int)cpc;
  out->math_warps = (int)mw;
  out->stages = stages;
  // 16 samples per block (squared and hinge losses): half as many hand-offs per sample; one CTA per SM
  int s16 = c->opt_stages > 0 ? std::min(c->opt_stages, 8) : 2;
  while (s16 >= 2 && Mma16Smem(s16, (size_t)cpc * 16, 2).total > kSmemBudget) --s16;
  out->stages16 = s16 >= 2 ? s16 : 0;
  const bool can16 = out->stages16 > 0;
  out->block = (c->opt_block_samples == 16 || (c->opt_block_samples == 0 && can16)) ? 16 : 8;
  if (out->block == 16 && !can16) return false;
  return true;
}

// ---- fp32 rows: the 16-sample cluster kernel with the Gram block on the fp32 pipes -------------------------------------
// A chain is spread over as many CTAs as idle SMs allow (a cluster of 2, 4 or 8), each with at most 64 chunks of 4
// columns: meant for few, wide chains that would otherwise hold one SM each.
constexpr int kF16Stages = 3;
bool f16_kernel_fits(const wpsgd_ctx* c, int nk, bool aligned, ClusterShape* out) {
  if (!aligned || (double)c->eta0 * (double)c->lambda > 0.25) return false;
  const long long chunks = c->d / 4;
  int C = c->opt_cluster;
  if (C <= 0) {
    C = 8;
    while (C > 1 && ((long long)nk * C > 148 || (chunks + C - 1) / C < 8)) C /= 2;
  }
  if (C != 1 && C != 2 && C != 4 && C != 8) return false;
  const long long cpc = (chunks + C - 1) / C;
  if (cpc < 1 || cpc > 64 || (long long)(C - 1) * cpc >= chunks) return false;
  if (Mma16Smem(kF16Stages, (size_t)cpc * 16, 3).total > kSmemBudget) return false;
  out->C = C;
  out->cpc = (int)cpc;
  out->math_warps = 8;
  out->stages16 = kF16Stages;
  out->block = 16;
  return true;
}

wpsgd_status launch_f16(wpsgd_ctx* c, const ChainParams& p, const ClusterShape& sh) {
  ClusterParams cp;
  cp.b.c = p;
  cp.b.stages = sh.stages16;
  cp.b.eta_lambda = (double)c->eta0 * (double)c->lambda;
  cp.b.spin_limit = c->opt_spin_limit;
  cp.b.drop_block = c->opt_drop_block;
  cp.b.group_order = nullptr;
  cp.chunks_per_cta = sh.cpc;
  const size_t smem = Mma16Smem(sh.stages16, (size_t)sh.cpc * 16, 3).total;
  auto go = [&](auto kern) -> wpsgd_status {
    CU_TRY(c, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(p.k * sh.C));
    cfg.blockDim = dim3((unsigned)(64 + 32 * sh.math_warps));
    cfg.dynamicSmemBytes = smem;
    cfg.stream = c->stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = (unsigned)sh.C;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    CU_TRY(c, cudaLaunchKernelEx(&cfg, kern, cp));
    c->launches++;
    return WPSGD_OK;
  };
  switch (c->loss) {
    case WPSGD_LOSS_HINGE: return go(chain_mma16_kernel<LOSS_HINGE, float>);
    case WPSGD_LOSS_LOGISTIC: return go(chain_mma16_kernel<LOSS_LOGISTIC, float>);
    default: return go(chain_mma16_kernel<LOSS_SQUARED, float>);
  }
}

wpsgd_status launch_mma(wpsgd_ctx* c, const ChainParams& p, const ClusterShape& sh) {
  ClusterParams cp;
  cp.b.c = p;
  cp.b.stages = sh.stages;
  cp.b.eta_lambda = (double)c->eta0 * (double)c->lambda;
  cp.b.spin_limit = c->opt_spin_limit;
  cp.b.drop_block = c->opt_drop_block;
  cp.b.group_order = nullptr;
  cp.chunks_per_cta = sh.cpc;
  const bool b16 = sh.block == 16;
  if (b16) cp.b.stages = sh.stages16;
  const size_t smem = b16 ? Mma16Smem(sh.stages16, (size_t)sh.cpc * 16, 2).total : MmaSmem(sh.stages, (size_t)sh.cpc * 16, MMA_SLOTS).total;
  auto go = [&](auto kern) -> wpsgd_status {
    CU_TRY(c, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(p.k * sh.C));
    cfg.blockDim = dim3((unsigned)(64 + 32 * sh.math_warps));
    cfg.dynamicSmemBytes = smem;
    cfg.stream = c->stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = (unsigned)sh.C;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    CU_TRY(c, cudaLaunchKernelEx(&cfg, kern, cp));
    c->launches++;
    return WPSGD_OK;
  };
  if (b16) {
    switch (c->loss) {
      case WPSGD_LOSS_HINGE: return go(chain_mma16_kernel<LOSS_HINGE, __nv_bfloat16>);
      case WPSGD_LOSS_LOGISTIC: return go(chain_mma16_kernel<LOSS_LOGISTIC, __nv_bfloat16>);
      default: return go(chain_mma16_kernel<LOSS_SQUARED, __nv_bfloat16>);
    }
  }
  switch (c->loss) {
    case WPSGD_LOSS_HINGE: return go(chain_mma_kernel<LOSS_HINGE, 4>);
    case WPSGD_LOSS_LOGISTIC: return go(chain_mma_kernel<LOSS_LOGISTIC, 4>);
    default: return go(chain_mma_kernel<LOSS_SQUARED, 4>);
  }
}

// Warp-per-node kernel: one CTA of four warps per SM, or two? A warp alone on its scheduler takes about 2640 cycles
// per block of 8 samples, two warps sharing one about 3000 each (measured, k = 1024, d = 256). With one CTA per SM
// there are 148 CTA slots and the remaining CTAs queue behind, longest first; with two there are 296 slots. Which
// finishes first depends on the step counts (equal work: 3.57 ms with two against 5.28 ms with one; speed ratio 16:
// 5.69 ms against 4.97 ms), so both schedules are played through on the host: CTAs in launch order (a CTA lasts as long
// as its longest chain) onto the slot that frees first.
bool two_warp_ctas_per_sm_finish_first(const std::vector<long long>& steps, int warps) {
  std::vector<long long> sorted(steps);
  std::sort(sorted.begin(), sorted.end(), [](long long a, long long b) { return a > b; });
  std::vector<long long> cta_cost;
  for (size_t i = 0; i < sorted.size(); i += (size_t)warps) cta_cost.push_back(sorted[i]);
  auto makespan = [&](int slots, double cycles_per_block) {
    std::vector<double> free_at((size_t)std::min<size_t>((size_t)slots, cta_cost.size()), 0.0);
    if (free_at.empty()) return 0.0;
    std::make_heap(free_at.begin(), free_at.end(), std::greater<double>());
    double end = 0.0;
    for (long long cost : cta_cost) {
      std::pop_heap(free_at.begin(), free_at.end(), std::greater<double>());
      const double t = free_at.back() + (double)cost * cycles_per_block;
      free_at.back() = t;
      end = std::max(end, t);
      std::push_heap(free_at.begin(), free_at.end(), std::greater<double>());
    }
    return end;
  };
  return makespan(2 * 148, 3000.0) < makespan(148, 2640.0);
}

// blocked kernel, one warp per node (small d)
template <typename XT>
bool block_warp_kernel_fits(const wpsgd_ctx* c, int nk, bool aligned, int* R_out, int* stages_out, int* warps_out) {
  constexpr int V = XVec<XT>::V;
  if (!aligned) return false;
  if ((double)c->eta0 * (double)c->lambda > 0.25) return false;
  const long long chunks = c->d / V;
  const int R = (int)((chunks + 31) / 32);
  if (R > 2) return false;
  const size_t row_bytes = (size_t)c->d * sizeof(XT);
  // Four nodes per CTA and two CTAs per SM. Each chain is bound by its own dependent instruction stream, so what
  // a long chain needs is few co-runners late in the run, not an equal share of work per SM: with chains dealt out
  // longest first, the CTAs of the longest chains land on the SMs first and are paired with the shortest ones.
  // (Measured on k = 1024, d = 256, speed ratio 4: 4.9 ms this way, 6.9 ms with one balanced 7-warp CTA per SM.)
  if (nk != c->k) return false;  // its node-to-CTA table covers the whole node set
  int warps = (int)std::min<long long>(4, std::max<long long>(1, nk));
  if (c->opt_threads >= 32 && c->opt_threads % 32 == 0) warps = std::min(BLKW_MAX_WARPS, c->opt_threads / 32);
  // one CTA per SM (a ring of 4 stages per warp takes the shared memory of a second one) or two (3 stages): see above
  const bool one_cta_per_sm = c->opt_stages >= 4 || (c->opt_stages == 0 && !two_warp_ctas_per_sm_finish_first(c->last_steps, warps));
  int stages = c->opt_stages > 0 ? std::min(c->opt_stages, 4) : (one_cta_per_sm ? 4 : 3);
  while (BlockWarpSmem(stages, row_bytes, warps).total > ((warps <= 4 && !one_cta_per_sm) ? 100 * 1024 : kSmemBudget)) {
    if (stages > 2) --stages;
    else if (warps > 1) --warps;
    else return false;
  }
  *R_out = R;
  *stages_out = stages;
  *warps_out = warps;
  return true;
}

// Nodes of every CTA of the warp-per-node kernel: longest first, consecutive ranks share a CTA; -1 fills the last one.
wpsgd_status upload_groups(wpsgd_ctx* c, const long long* n_steps_host, int warps, int* ctas_out) {
  const int k = c->k;
  const int ctas = (k + warps - 1) / warps;
  std::vector<int> group((size_t)ctas * warps, -1);
  std::iota(group.begin(), group.begin() + k, 0);
  std::stable_sort(group.begin(), group.begin() + k, [&](int a, int b) { return n_steps_host[a] > n_steps_host[b]; });
  CU_TRY(c, cudaMemcpyAsync(c->t_group, group.data(), group.size() * sizeof(int), cudaMemcpyHostToDevice, c->stream));
  *ctas_out = ctas;
  return WPSGD_OK;
}

template <typename XT, int R>
wpsgd_status launch_block_warp_r(wpsgd_ctx* c, const BlockParams& bp, size_t smem, int ctas, int warps) {
  auto go = [&](auto kern) -> wpsgd_status {
    CU_TRY(c, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    kern<<<ctas, 32 * warps, smem, c->stream>>>(bp);
    CU_TRY(c, cudaGetLastError());
    c->launches++;
    return WPSGD_OK;
  };
  const bool decay = c->sched == WPSGD_LR_INV_SQRT;
  switch (c->loss) {
    case WPSGD_LOSS_HINGE: return decay ? go(chain_block_warp_kernel<XT, R, LOSS_HINGE, true>) : go(chain_block_warp_kernel<XT, R, LOSS_HINGE, false>);
    case WPSGD_LOSS_LOGISTIC: return decay ? go(chain_block_warp_kernel<XT, R, LOSS_LOGISTIC, true>) : go(chain_block_warp_kernel<XT, R, LOSS_LOGISTIC, false>);
    default: return decay ? go(chain_block_warp_kernel<XT, R, LOSS_SQUARED, true>) : go(chain_block_warp_kernel<XT, R, LOSS_SQUARED, false>);
  }
}

template <typename XT>
wpsgd_status launch_block_warp(wpsgd_ctx* c, const ChainParams& p, int R, int stages, int warps) {
  BlockParams bp;
  bp.c = p;
  bp.stages = stages;
  bp.eta_lambda = (double)c->eta0 * (double)c->lambda;
  bp.spin_limit = c->opt_spin_limit;
  bp.drop_block = -1;
  bp.group_order = c->t_group;
  int ctas = 0;
  wpsgd_status s = upload_groups(c, c->last_steps.data(), warps, &ctas);
  if (s != WPSGD_OK) return s;
  const size_t smem = BlockWarpSmem(stages, (size_t)c->d * sizeof(XT), warps).total;
  return R == 1 ? launch_block_warp_r<XT, 1>(c, bp, smem, ctas, warps) : launch_block_warp_r<XT, 2>(c, bp, smem, ctas, warps);
}

template <typename XT>
wpsgd_status launch_dense(wpsgd_ctx* c, const ChainParams& p) {
  constexpr int V = XVec<XT>::V;
  const long long d = c->d;
  const bool aligned = ((uintptr_t)p.X % 16 == 0) && ((p.ld * (long long)sizeof(XT)) % 16 == 0) && (d % V == 0) &&
                       ((uintptr_t)c->W % 16 == 0);
  const long long chunks = d / V;
  int variant = c->opt_variant;
  int bthreads = 0, bR = 0, bstages = 0;
  const bool block_ok = block_kernel_fits<XT>(c, aligned, &bthreads, &bR, &bstages);
  int wR = 0, wstages = 0, wwarps = 0;
  const bool block_warp_ok = block_warp_kernel_fits<XT>(c, p.k, aligned, &wR, &wstages, &wwarps);
  ClusterShape mma_shape, f16_shape;
  const bool mma_ok = sizeof(XT) == 2 && mma_kernel_fits(c, aligned, &mma_shape);
  const bool f16_ok = sizeof(XT) == 4 && f16_kernel_fits(c, p.k, aligned, &f16_shape);
  if (variant == 0) {
    if (!aligned) variant = 1;
    else if (f16_ok && f16_shape.C >= 4 && chunks >= 128) variant = 9;  // few wide fp32 chains: spread each over idle SMs
    else if (chunks <= 64) variant = block_warp_ok ? 5 : 3;
    else if (sizeof(XT) == 2 && chunks >= 256 && mma_ok) variant = 8;  // wide bf16 rows: tensor-core cluster kernel
    else if (block_ok) variant = 4;
    else variant = (chunks > 512 * 4) ? 1 : 2;
  }
  if (variant == 5) {
    if (!block_warp_ok)
      return fail(c, WPSGD_ERR_UNSUPPORTED,
                  "blocked warp kernel needs 16-byte aligned rows of at most 64 chunks, "
                  "eta*lambda <= 0.25");
    return launch_block_warp<XT>(c, p, wR, wstages, wwarps);
  }
  if (variant == 8) {
    ClusterShape sh;
    if (sizeof(XT) != 2 || !mma_kernel_fits(c, aligned, &sh))
      return fail(c, WPSGD_ERR_UNSUPPORTED,
                  "tensor-core cluster kernel needs bf16 rows, 16-byte aligned, eta*lambda <= 0.25, a "
                  "cluster of 1, 2, 4 or 8 CTAs with at most 256 chunks of a row each and at most 16 math warps in all");
    return launch_mma(c, p, sh);
  }
  if (variant == 9) {
    if (!f16_ok)
      return fail(c, WPSGD_ERR_UNSUPPORTED,
                  "16-sample cluster kernel for fp32 rows needs 16-byte aligned rows, eta*lambda <= 0.25 and a cluster of "
                  "1, 2, 4 or 8 CTAs with at most 64 chunks of a row each");
    return launch_f16(c, p, f16_shape);
  }
  if (variant == 4) {
    if (!block_ok)
      return fail(c, WPSGD_ERR_UNSUPPORTED,
                  "blocked kernel needs 16-byte aligned rows of at most 8 KiB and eta*lambda <= 0.25");
    return launch_block<XT>(c, p, bthreads, bR, bstages);
  }
  if ((variant == 2 || variant == 3) && !aligned)
    return fail(c, WPSGD_ERR_UNSUPPORTED, "register kernels need 16-byte aligned rows and d a multiple of 16 bytes");
  if (variant == 3 && chunks > 32 * 4) return fail(c, WPSGD_ERR_UNSUPPORTED, "warp-per-node kernel: d too large");
  if (variant == 2 && chunks > 512 * 4) return fail(c, WPSGD_ERR_UNSUPPORTED, "CTA-per-node kernel: d too large");
  if (variant == 1) {
    chain_generic_kernel<XT><<<p.k, 256, 0, c->stream>>>(p);
    CU_TRY(c, cudaGetLastError());
    c->launches++;
    return WPSGD_OK;
  }
  if (variant != 2 && variant != 3) return fail(c, WPSGD_ERR_UNSUPPORTED, "dense_variant not available");
  int threads = 32, R = 1;
  if (variant == 3) {
    R = (int)((chunks + 31) / 32);
  } else {
    threads = c->opt_threads > 0 ? c->opt_threads : (int)std::min<long long>(512, ((chunks + 31) / 32) * 32);
    R = (int)((chunks + threads - 1) / threads);
  }
  if (R > 2) R = 4;  // instantiated: 1, 2, 4
  if ((long long)R * threads < chunks) return fail(c, WPSGD_ERR_UNSUPPORTED, "threads too few for d");
  int pf = c->opt_prefetch > 0 ? c->opt_prefetch : std::max(2, 8 / R);
  pf = pf >= 8 ? 8 : (pf >= 4 ? 4 : 2);
  const bool bpn = variant == 2;
  switch (R) {
    case 1: return launch_reg_pf<XT, 1>(c, p, bpn, threads, pf);
    case 2: return launch_reg_pf<XT, 2>(c, p, bpn, threads, pf);
    default: return launch_reg_pf<XT, 4>(c, p, bpn, threads, pf);
  }
}

// Nodes launched together (a run of `count` consecutive entries of the longest-first order) once `ready` has happened.
struct LaunchGroup {
  int count;
  cudaEvent_t ready;
};

wpsgd_status run_dense_common(wpsgd_ctx* c, const void* X, wpsgd_xtype xt, long long ld, const float* y,
                              const long long* shard_off, const long long* n_steps, const float* w0, bool resume,
                              const std::vector<LaunchGroup>* groups = nullptr) {
  if (xt != WPSGD_X_F32 && xt != WPSGD_X_BF16) return fail(c, WPSGD_ERR_INVALID_ARG, "unknown feature type");
  if (ld < c->d) return fail(c, WPSGD_ERR_INVALID_ARG, "ld_elems < d");
  Plan pl;
  std::vector<long long> first = resume ? c->steps_done : std::vector<long long>(c->k, 0);
  wpsgd_status s = make_plan(c, (const long long*)shard_off, (const long long*)n_steps, first, &pl);
  if (s != WPSGD_OK) return s;
  if (pl.total > 0 && (!X || !y)) return fail(c, WPSGD_ERR_INVALID_ARG, "X or y is NULL");
  s = upload_plan_and_stream(c, pl);
  if (s != WPSGD_OK) return s;
  c->last_steps = pl.steps;
  ChainParams p;
  p.X = X; p.ld = ld; p.y = y;
  p.shard_off = c->t_shard_off; p.n_steps = c->t_steps; p.first = c->t_first; p.idx_off = c->t_idx_off;
  p.idx = c->idx; p.order = c->t_order; p.W = c->W; p.w0 = w0; p.resume = resume ? 1 : 0;
  p.k = c->k; p.d = c->d; p.eta0 = c->eta0; p.sched = c->sched; p.lambda = c->lambda; p.loss = c->loss;
  p.status = c->status;
  s = timing_begin(c);
  if (s != WPSGD_OK) return s;
  if (!groups) {
    s = (xt == WPSGD_X_F32) ? launch_dense<float>(c, p) : launch_dense<__nv_bfloat16>(c, p);
    if (s != WPSGD_OK) return s;
  } else {
    // one launch per group of nodes, each behind the event that says its rows are on the device
    int first_slot = 0;
    for (const LaunchGroup& g : *groups) {
      CU_TRY(c, cudaStreamWaitEvent(c->stream, g.ready, 0));
      if (g.count > 0) {
        ChainParams q = p;
        q.order = c->t_order + first_slot;
        q.k = g.count;
        s = (xt == WPSGD_X_F32) ? launch_dense<float>(c, q) : launch_dense<__nv_bfloat16>(c, q);  // grids follow q.k
        if (s != WPSGD_OK) return s;
      }
      first_slot += g.count;
    }
  }
  s = timing_end(c);
  if (s != WPSGD_OK) return s;
  for (int j = 0; j < c->k; ++j) c->steps_done[j] = first[j] + n_steps[j];
  c->have_run = true;
  c->scaled = false;
  return WPSGD_OK;
}

// ---- sparse chain launch ---------------------------------------------------------------------------------
wpsgd_status run_csr_common(wpsgd_ctx* c, const long long* row_ptr, const int* col_idx, const float* val, const float* y,
                            const long long* shard_off, const long long* n_steps, const float* w0, bool resume) {
  Plan pl;
  std::vector<long long> first = resume ? c->steps_done : std::vector<long long>(c->k, 0);
  wpsgd_status s = make_plan(c, shard_off, n_steps, first, &pl);
  if (s != WPSGD_OK) return s;
  if (pl.total > 0 && (!row_ptr || !col_idx || !val || !y)) return fail(c, WPSGD_ERR_INVALID_ARG, "a CSR array or y is NULL");
  s = upload_plan_and_stream(c, pl);
  if (s != WPSGD_OK) return s;
  if (!resume || !c->scaled) {
    // fresh chains start from w0 with scale 1; chains continued from a dense run keep their models and get scale 1
    csr_init_kernel<<<grid_for((long long)c->k * c->d, 256), 256, 0, c->stream>>>(c->W, c->scale, w0, c->k, c->d, resume ? 1 : 0);
    CU_TRY(c, cudaGetLastError());
    c->launches++;
  }
  CsrParams p;
  p.row_ptr = row_ptr; p.col_idx = col_idx; p.val = val; p.y = y;
  p.shard_off = c->t_shard_off; p.n_steps = c->t_steps; p.first = c->t_first; p.idx_off = c->t_idx_off; p.idx = c->idx;
  p.order = c->t_order; p.U = c->W; p.scale = c->scale; p.k = c->k; p.d = c->d;
  p.eta0 = c->eta0; p.sched = c->sched; p.lambda = c->lambda; p.loss = c->loss; p.resume = resume ? 1 : 0;
  p.status = c->status;
  s = timing_begin(c);
  if (s != WPSGD_OK) return s;
  if (c->opt_sparse_variant == 1) {
    const int pf = c->opt_prefetch > 0 ? c->opt_prefetch : 4;
    if (pf >= 8) chain_csr_kernel<8><<<c->k, 32, 0, c->stream>>>(p);
    else if (pf >= 4) chain_csr_kernel<4><<<c->k, 32, 0, c->stream>>>(p);
    else chain_csr_kernel<2><<<c->k, 32, 0, c->stream>>>(p);
    CU_TRY(c, cudaGetLastError());
  } else {
    const size_t smem = sizeof(CsrBlockSmem);
    auto go = [&](auto kern) -> wpsgd_status {
      CU_TRY(c, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
      kern<<<c->k, CSRB_THREADS, smem, c->stream>>>(p);
      CU_TRY(c, cudaGetLastError());
      return WPSGD_OK;
    };
    switch (c->loss) {
      case WPSGD_LOSS_HINGE: s = go(chain_csr_block_kernel<LOSS_HINGE>); break;
      case WPSGD_LOSS_LOGISTIC: s = go(chain_csr_block_kernel<LOSS_LOGISTIC>); break;
      default: s = go(chain_csr_block_kernel<LOSS_SQUARED>); break;
    }
    if (s != WPSGD_OK) return s;
  }
  c->launches++;
  s = timing_end(c);
  if (s != WPSGD_OK) return s;
  for (int j = 0; j < c->k; ++j) c->steps_done[j] = first[j] + n_steps[j];
  c->have_run = true;
  c->scaled = true;
  return WPSGD_OK;
}

}  // namespace

// ---- built-in scratch of the entry point that allocates nothing ----------------------------------------
// Layout inside one file-scope device array (every section 256-byte aligned). The array exists once per
// GPU that loads this library and lives until the process exits.
namespace {
constexpr size_t align256(size_t x) { return (x + 255) / 256 * 256; }
struct StaticLayout {
  size_t W = 0;
  size_t idx = align256(W + sizeof(float) * (size_t)WPSGD_STATIC_MAX_MODEL_ELEMS);
  size_t shard_off = align256(idx + sizeof(uint32_t) * ((size_t)WPSGD_STATIC_MAX_STEPS + 64 * WPSGD_STATIC_MAX_NODES));
  size_t steps = align256(shard_off + sizeof(long long) * (WPSGD_STATIC_MAX_NODES + 1));
  size_t first = align256(steps + sizeof(long long) * WPSGD_STATIC_MAX_NODES);
  size_t idx_off = align256(first + sizeof(long long) * WPSGD_STATIC_MAX_NODES);
  size_t rows = align256(idx_off + sizeof(long long) * (WPSGD_STATIC_MAX_NODES + 1));
  size_t count = align256(rows + sizeof(long long) * WPSGD_STATIC_MAX_NODES);
  size_t order = align256(count + sizeof(long long) * WPSGD_STATIC_MAX_NODES);
  size_t ids = align256(order + sizeof(int) * WPSGD_STATIC_MAX_NODES);
  size_t group = align256(ids + sizeof(int) * WPSGD_STATIC_MAX_NODES);
  size_t weights = align256(group + sizeof(int) * (WPSGD_STATIC_MAX_NODES + 8));
  size_t scale = align256(weights + sizeof(double) * WPSGD_STATIC_MAX_NODES);
  size_t status = align256(scale + sizeof(double) * WPSGD_STATIC_MAX_NODES);
  size_t total = align256(status + sizeof(DevStatus));
};
constexpr size_t kStaticBytes = align256(sizeof(float) * (size_t)WPSGD_STATIC_MAX_MODEL_ELEMS) +
                                align256(sizeof(uint32_t) * ((size_t)WPSGD_STATIC_MAX_STEPS + 64 * WPSGD_STATIC_MAX_NODES)) +
                                13 * align256(sizeof(long long) * (WPSGD_STATIC_MAX_NODES + 1));
constexpr int kStaticMaxDevices = 64;
}  // namespace

static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

namespace {
// In host code the name g_static_scratch is only a handle of the symbol, not a device address; the address
// a kernel can use comes from cudaGetSymbolAddress, asked once per device with that device current.
unsigned char* g_static_base[kStaticMaxDevices] = {nullptr};

wpsgd_status static_scratch_base(int device, unsigned char** out) {
  static_assert(sizeof(DevStatus) <= 256, "status word must fit its section");
  if (StaticLayout().total > kStaticBytes) return fail(nullptr, WPSGD_ERR_STATE, "built-in scratch layout exceeds the array");
  if (!g_static_base[device]) {
    void* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess || !p) {
      cudaGetLastError();
      return fail(nullptr, WPSGD_ERR_CUDA, std::string("cudaGetSymbolAddress(built-in scratch): ") + cudaGetErrorString(e));
    }
    g_static_base[device] = (unsigned char*)p;
  }
  *out = g_static_base[device];
  return WPSGD_OK;
}
}  // namespace

extern "C" {

wpsgd_status wpsgd_create(int device, void* cuda_stream, int32_t k, int64_t d, wpsgd_ctx** out) {
  if (!out) return fail(nullptr, WPSGD_ERR_INVALID_ARG, "out is NULL");
  *out = nullptr;
  if (k < 1 || d < 1) return fail(nullptr, WPSGD_ERR_INVALID_ARG, "k and d must be >= 1");
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) {
    cudaGetLastError();
    return fail(nullptr, WPSGD_ERR_CUDA, "no CUDA device available");
  }
  if (device < 0 || device >= ndev) return fail(nullptr, WPSGD_ERR_INVALID_ARG, "device index out of range");
  DeviceGuard guard(device);
  wpsgd_ctx* c = new wpsgd_ctx();
  c->device = device;
  c->stream = (cudaStream_t)cuda_stream;
  c->k = k;
  c->d = d;
  c->steps_done.assign(k, 0);
  c->node_ids.resize(k);
  std::iota(c->node_ids.begin(), c->node_ids.end(), 0);
  auto bail = [&](cudaError_t e, const char* what) {
    g_err = std::string(what) + ": " + cudaGetErrorString(e);
    const wpsgd_status s = (e == cudaErrorMemoryAllocation) ? WPSGD_ERR_ALLOC : WPSGD_ERR_CUDA;
    cudaGetLastError();
    wpsgd_destroy(c);
    return s;
  };
  cudaError_t e;
#define ALLOC(ptr, bytes)                                         \
  if ((e = cudaMalloc((void**)&(ptr), (bytes))) != cudaSuccess) return bail(e, "cudaMalloc(" #ptr ")");
  ALLOC(c->W, (size_t)k * (size_t)d * sizeof(float));
  ALLOC(c->scale, (size_t)k * sizeof(double));
  ALLOC(c->t_shard_off, (size_t)(k + 1) * sizeof(long long));
  ALLOC(c->t_steps, (size_t)k * sizeof(long long));
  ALLOC(c->t_first, (size_t)k * sizeof(long long));
  ALLOC(c->t_idx_off, (size_t)(k + 1) * sizeof(long long));
  ALLOC(c->t_rows, (size_t)k * sizeof(long long));
  ALLOC(c->t_count, (size_t)k * sizeof(long long));
  ALLOC(c->t_order, (size_t)k * sizeof(int));
  ALLOC(c->t_ids, (size_t)k * sizeof(int));
  ALLOC(c->t_group, ((size_t)k + 8) * sizeof(int));
  ALLOC(c->t_weights, (size_t)k * sizeof(double));
  ALLOC(c->status, sizeof(DevStatus));
#undef ALLOC
  if ((e = cudaMemsetAsync(c->status, 0, sizeof(DevStatus), c->stream)) != cudaSuccess) return bail(e, "cudaMemsetAsync");
  *out = c;
  return WPSGD_OK;
}

wpsgd_status wpsgd_destroy(wpsgd_ctx* c) {
  if (!c) return WPSGD_OK;
  DeviceGuard guard(c->device);
  cudaStreamSynchronize(c->stream);
  void* ptrs[] = {c->W, c->scale, c->t_shard_off, c->t_steps, c->t_first, c->t_idx_off, c->t_rows, c->t_count, c->t_order,
                  c->t_ids, c->t_group, c->t_weights, c->idx, c->status, c->part, c->st_X, c->st_y, c->st_v, c->st_w0, c->st_rp, c->st_ci, c->st_va};
  for (void* p : ptrs)
    if (p) cudaFree(p);
  if (c->ev0) cudaEventDestroy(c->ev0);
  if (c->ev1) cudaEventDestroy(c->ev1);
  if (c->ev_fork) cudaEventDestroy(c->ev_fork);
  for (cudaEvent_t e : c->ev_group)
    if (e) cudaEventDestroy(e);
  if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
  cudaGetLastError();
  delete c;
  return WPSGD_OK;
}

wpsgd_status wpsgd_set_option(wpsgd_ctx* c, const char* name, int64_t value) {
  if (!c || !name) return fail(c, WPSGD_ERR_INVALID_ARG, "ctx or name is NULL");
  const std::string n(name);
  if (n == "dense_variant") {
    if (value < 0 || value > 9 || value == 6 || value == 7) return fail(c, WPSGD_ERR_INVALID_ARG, "dense_variant must be 0..5, 8 or 9");
    c->opt_variant = (int)value;
  } else if (n == "prefetch") {
    if (value < 0 || value > 64) return fail(c, WPSGD_ERR_INVALID_ARG, "prefetch must be 0..64");
    c->opt_prefetch = (int)value;
  } else if (n == "threads") {
    if (value != 0 && (value < 32 || value > 512 || value % 32)) return fail(c, WPSGD_ERR_INVALID_ARG, "threads must be 0 or a multiple of 32 in 32..512");
    c->opt_threads = (int)value;
  } else if (n == "cluster") {
    if (value != 0 && value != 1 && value != 2 && value != 4 && value != 8) return fail(c, WPSGD_ERR_INVALID_ARG, "cluster must be 0, 1, 2, 4 or 8");
    c->opt_cluster = (int)value;
  } else if (n == "host_pipeline") {
    if (value != 0 && value != 1) return fail(c, WPSGD_ERR_INVALID_ARG, "host_pipeline must be 0 or 1");
    c->opt_host_pipeline = (int)value;
  } else if (n == "block_samples") {
    if (value != 0 && value != 8 && value != 16) return fail(c, WPSGD_ERR_INVALID_ARG, "block_samples must be 0, 8 or 16");
    c->opt_block_samples = (int)value;
  } else if (n == "sparse_variant") {
    if (value < 0 || value > 2) return fail(c, WPSGD_ERR_INVALID_ARG, "sparse_variant must be 0, 1 or 2");
    c->opt_sparse_variant = (int)value;
  } else if (n == "stages") {
    if (value < 0 || value == 1 || value > 8) return fail(c, WPSGD_ERR_INVALID_ARG, "stages must be 0 or 2..8");
    c->opt_stages = (int)value;
  } else if (n == "timing") {
    if (value != 0 && value != 1) return fail(c, WPSGD_ERR_INVALID_ARG, "timing must be 0 or 1");
    c->opt_timing = (int)value;
  } else if (n == "sampling") {
    if (value != 0 && value != 1) return fail(c, WPSGD_ERR_INVALID_ARG, "sampling must be 0 (i.i.d. draws) or 1 (shuffled order)");
    c->opt_sampling = (int)value;
  } else if (n == "test_drop_block") {
    c->opt_drop_block = value;
  } else if (n == "spin_limit") {
    if (value < 1) return fail(c, WPSGD_ERR_INVALID_ARG, "spin_limit must be >= 1");
    c->opt_spin_limit = value;
  } else {
    return fail(c, WPSGD_ERR_INVALID_ARG, "unknown option: " + n);
  }
  return WPSGD_OK;
}

wpsgd_status wpsgd_set_node_ids(wpsgd_ctx* c, const int32_t* ids) {
  if (!c) return fail(nullptr, WPSGD_ERR_INVALID_ARG, "ctx is NULL");
  if (!ids) {
    std::iota(c->node_ids.begin(), c->node_ids.end(), 0);
    return WPSGD_OK;
  }
  for (int j = 0; j < c->k; ++j)
    if (ids[j] < 0) return fail(c, WPSGD_ERR_INVALID_ARG, "node ids must be >= 0");
  c->node_ids.assign(ids, ids + c->k);
  return WPSGD_OK;
}

wpsgd_status wpsgd_run(wpsgd_ctx* c, const void* X, wpsgd_xtype xt, int64_t ld_elems, const float* y,
                       const int64_t* shard_off, const int64_t* n_steps, float eta0, wpsgd_lr sched, float lambda,
                       wpsgd_loss loss, uint64_t seed, const float* w0) {
  if (!c) return fail(nullptr, WPSGD_ERR_INVALID_ARG, "ctx is NULL");
  DeviceGuard guard(c->device);
  wpsgd_status s = check_hyper(c, eta0, (int)sched, lambda, (int)loss);
  if (s != WPSGD_OK) return s;
  c->eta0 = eta0; c->sched = (int)sched; c->lambda = lambda; c->loss = (int)loss; c->seed = seed;
  c->have_run = false;
  return run_dense_common(c, X, xt, ld_elems, y, (const long long*)shard_off, (const long long*)n_steps, w0, false);
}

wpsgd_status wpsgd_continue(wpsgd_ctx* c, const void* X, wpsgd_xtype xt, int64_t ld_elems, const float* y,
                            const int64_t* shard_off, const int64_t* n_more) {
  if (!c) return fail(nullptr, WPSGD_ERR_INVALID_ARG, "ctx is NULL");
  if (!c->have_run) return fail(c, WPSGD_ERR_STATE, "continue before run");
  if (c->scaled) return fail(c, WPSGD_ERR_UNSUPPORTED, "chains started on CSR rows continue with wpsgd_continue_csr");
  DeviceGuard guard(c->device);
  return run_dense_common(c, X, xt, ld_elems, y, (const long long*)shard_off, (const long long*)n_more, nullptr, true);
}

wpsgd_status wpsgd_run_csr(wpsgd_ctx* c, const int64_t* row_ptr, const int32_t* col_idx, const float* val,
                           const float* y, const int64_t* shard_off, const int64_t* n_steps, float eta0,
                           wpsgd_lr sched, float lambda, wpsgd_loss loss, uint64_t seed, const float* w0) {
  if (!c) return fail(nullptr, WPSGD_ERR_INVALID_ARG, "ctx is NULL");
  DeviceGuard guard(c->device);
  wpsgd_status s = check_hyper(c, eta0, (int)sched, lambda, (int)loss);
  if (s != WPSGD_OK) return s;
  c->eta0 = eta0; c->sched = (int)sched; c->lambda = lambda; c->loss = (int)loss; c->seed = seed;
  c->have_run = false;
  return run_csr_common(c, (const long long*)row_ptr, col_idx, val, y, (const long long*)shard_off,
                        (const long long*)n_steps, w0, false);
}

wpsgd_status wpsgd_continue_csr(wpsgd_ctx* c, const int64_t* row_ptr, const int32_t* col_idx, const float* val,
                                const float* y, const int64_t* shard_off, const int64_t* n_more) {
  if (!c) return fail(nullptr, WPSGD_ERR_INVALID_ARG, "ctx is NULL");
  if (!c->have_run) return fail(c, WPSGD_ERR_STATE, "continue before run");
  DeviceGuard guard(c->device);
  return run_csr_common(c, (const long long*)row_ptr, col_idx, val, y, (const long long*)shard_off,
                        (const long long*)n_more, nullptr, true);
}

wpsgd_status wpsgd_get_weights(wpsgd_ctx* c, double r, double* weights, int* cond_holds) {
  if (!c) return fail(nullptr, WPSGD_ERR_INVALID_ARG, "ctx is NULL");
  if (!c->have_run) return fail(c, WPSGD_ERR_STATE, "weights before run");
  std::string why;
  wpsgd_status s = weights_host(c->steps_done.data(), c->k, c->eta0, c->sched, c->lambda, r, weights, cond_holds, nullptr, &why);
  return s == WPSGD_OK ? s : fail(c, s, why);
}

wpsgd_status wpsgd_weights(const int64_t* n_steps, int32_t k, float eta0, wpsgd_lr sched, float lambda, double r,
                           double* weights, int* cond_holds, double* sum_rT) {
  std::string why;
  wpsgd_status s = weights_host((const long long*)n_steps, k, eta0, (int)sched, lambda, r, weights, cond_holds, sum_rT, &why);
  return s == WPSGD_OK ? s : fail(nullptr, s, why);
}

wpsgd_status wpsgd_span_valid(const int64_t* n_steps, int32_t k, float eta0, float lambda, double r, int64_t span,
                              double* lhs, int* holds) {
  if (span < 0) return fail(nullptr, WPSGD_ERR_INVALID_ARG, "span_valid: span must be >= 0");
  if (!((double)eta0 * (double)lambda < 1.0) || !(eta0 >= 0.0f) || !(lambda >= 0.0f))
    return fail(nullptr, WPSGD_ERR_INVALID_ARG, "span_valid: need eta0 >= 0, lambda >= 0, eta0 * lambda < 1");
  if (!n_steps || k < 1) return fail(nullptr, WPSGD_ERR_INVALID_ARG, "span_valid: null argument or k < 1");
  std::string why;
  std::vector<double> lg;
  wpsgd_status s = log_rates((const long long*)n_steps, k, (double)eta0, WPSGD_LR_CONST, (double)lambda, r, &lg, &why);
  if (s != WPSGD_OK) return fail(nullptr, s, why);
  // log of sum_j r^{T_j}, summed from the largest term
  const double mx = *std::max_element(lg.begin(), lg.end());
  double tot = 0.0;
  for (int j = 0; j < k; ++j) tot += std::exp(lg[j] - mx);
  const double log_lhs = std::log((double)k) - (mx + std::log(tot)) + (double)span * std::log1p(-(double)eta0 * (double)lambda);
  const double v = std::exp(log_lhs);
  if (lhs) *lhs = v;
  if (holds) *holds = log_lhs < 0.0 ? 1 : 0;
  return WPSGD_OK;
}

wpsgd_status wpsgd_sample_indices_host(uint64_t seed, int32_t node, int64_t m, int64_t n_begin, int64_t count,
                                       int32_t sampling, uint32_t* out) {
  if (node < 0 || m < 1 || m > 0xFFFFFFFFll || n_begin < 0 || count < 0 || (sampling != 0 && sampling != 1))
    return fail(nullptr, WPSGD_ERR_INVALID_ARG,
                "sample_indices_host: need node >= 0, 1 <= m < 2^32, n_begin >= 0, count >= 0, sampling 0 or 1");
  if (count == 0) return WPSGD_OK;
  if (!out) return fail(nullptr, WPSGD_ERR_INVALID_ARG, "out is NULL");
  emit_indices(sampling, seed, (uint32_t)node, n_begin, count, (uint32_t)m, out, 0, 1);  // the kernels' own function
  return WPSGD_OK;
}

wpsgd_status wpsgd_validate_csr(wpsgd_ctx* c, const int64_t* row_ptr, const int32_t* col_idx, int64_t n_rows, int64_t nnz) {
  if (!c) return fail(nullptr, WPSGD_ERR_INVALID_ARG, "ctx is NULL");
  if (n_rows < 0 || nnz < 0 || !row_ptr || (nnz > 0 && !col_idx)) return fail(c, WPSGD_ERR_INVALID_ARG, "validate_csr: bad argument");
  if (n_rows == 0) return WPSGD_OK;
  DeviceGuard guard(c->device);
  validate_csr_kernel<<<grid_for(n_rows, 8), 256, 0, c->stream>>>((const long long*)row_ptr, col_idx, n_rows, nnz, c->d, c->status);
  CU_TRY(c, cudaGetLastError());
  c->launches++;
  return WPSGD_OK;
}

wpsgd_status wpsgd_combine(wpsgd_ctx* c, double r, float* v_out) {
  if (!c) return fail(nullptr, WPSGD_ERR_INVALID_ARG, "ctx is NULL");
  if (!c->have_run) return fail(c, WPSGD_ERR_STATE, "combine before run");
  if (!v_out) return fail(c, WPSGD_ERR_INVALID_ARG, "v_out is NULL");
  DeviceGuard guard(c->device);
  std::vector<double> w(c->k);
  std::string why;
  wpsgd_status s = weights_host(c->steps_done.data(), c->k, c->eta0, c->sched, c->lambda, r, w.data(), nullptr, nullptr, &why);
  if (s != WPSGD_OK) return fail(c, s, why);
  CU_TRY(c, cudaMemcpyAsync(c->t_weights, w.data(), c->k * sizeof(double), cudaMemcpyHostToDevice, c->stream));
  combine_kernel<<<grid_for(c->d, 256), 256, 0, c->stream>>>(c->W, c->t_weights, c->scaled ? c->scale : nullptr, c->k,
                                                            c->d, v_out);
  CU_TRY(c, cudaGetLastError());
  c->launches++;
  return WPSGD_OK;
}

wpsgd_status wpsgd_combine_weighted(wpsgd_ctx* c, const double* weights, float* v_out) {
  if (!c) return fail(nullptr, WPSGD_ERR_INVALID_ARG, "ctx is NULL");
  if (!c->have_run) return fail(c, WPSGD_ERR_STATE, "combine before run");
  if (!v_out || !weights) return fail(c, WPSGD_ERR_INVALID_ARG, "weights or v_out is NULL");
  for (int j = 0; j < c->k; ++j)
    if (!std::isfinite(weights[j])) return fail(c, WPSGD_ERR_INVALID_ARG, "a weight is not finite");
  DeviceGuard guard(c->device);
  CU_TRY(c, cudaMemcpyAsync(c->t_weights, weights, c->k * sizeof(double), cudaMemcpyHostToDevice, c->stream));
  combine_kernel<<<grid_for(c->d, 256), 256, 0, c->stream>>>(c->W, c->t_weights, c->scaled ? c->scale : nullptr, c->k,
                                                            c->d, v_out);
  CU_TRY(c, cudaGetLastError());
  c->launches++;
  return WPSGD_OK;
}

wpsgd_status wpsgd_last_chain_ms(wpsgd_ctx* c, float* ms) {
  if (!c || !ms) return fail(c, WPSGD_ERR_INVALID_ARG, "ctx or ms is NULL");
  if (!c->ev_valid) return fail(c, WPSGD_ERR_STATE, "no timed chain launch (set option \"timing\" to 1 before the run)");
  DeviceGuard guard(c->device);
  CU_TRY(c, cudaEventSynchronize(c->ev1));
  CU_TRY(c, cudaEventElapsedTime(ms, c->ev0, c->ev1));
  return WPSGD_OK;
}

wpsgd_status wpsgd_get_models(wpsgd_ctx* c, float* W_out) {
  if (!c) return fail(nullptr, WPSGD_ERR_INVALID_ARG, "ctx is NULL");
  if (!c->have_run) return fail(c, WPSGD_ERR_STATE, "get_models before run");
  if (!W_out) return fail(c, WPSGD_ERR_INVALID_ARG, "W_out is NULL");
  DeviceGuard guard(c->device);
  export_models_kernel<<<grid_for((long long)c->k * c->d, 256), 256, 0, c->stream>>>(
      c->W, c->scaled ? c->scale : nullptr, c->k, c->d, W_out);
  CU_TRY(c, cudaGetLastError());
  c->launches++;
  return WPSGD_OK;
}

wpsgd_status wpsgd_set_models(wpsgd_ctx* c, const float* v) {
  if (!c) return fail(nullptr, WPSGD_ERR_INVALID_ARG, "ctx is NULL");
  if (!c->have_run) return fail(c, WPSGD_ERR_STATE, "set_models before run");
  if (!v) return fail(c, WPSGD_ERR_INVALID_ARG, "v is NULL");
  DeviceGuard guard(c->device);
  broadcast_model_kernel<<<grid_for((long long)c->k * c->d, 256), 256, 0, c->stream>>>(c->W, c->scale, v, c->k, c->d);
  CU_TRY(c, cudaGetLastError());
  c->launches++;
  return WPSGD_OK;
}

wpsgd_status wpsgd_sample_indices(wpsgd_ctx* c, uint64_t seed, int32_t node, int64_t m, int64_t n_begin, int64_t count,
                                  uint32_t* out) {
  if (!c) return fail(nullptr, WPSGD_ERR_INVALID_ARG, "ctx is NULL");
  if (node < 0 || m < 1 || m > 0xFFFFFFFFll || n_begin < 0 || count < 0)
    return fail(c, WPSGD_ERR_INVALID_ARG, "sample_indices: need node >= 0, 1 <= m < 2^32, n_begin >= 0, count >= 0");
  if (count == 0) return WPSGD_OK;
  if (!out) return fail(c, WPSGD_ERR_INVALID_ARG, "out is NULL");
  DeviceGuard guard(c->device);
  index_single_kernel<<<grid_for(c->opt_sampling ? count : (count + 3) / 4 + 1, 256), 256, 0, c->stream>>>(c->opt_sampling, seed, node, m, n_begin, count, out);
  CU_TRY(c, cudaGetLastError());
  c->launches++;
  return WPSGD_OK;
}

wpsgd_status wpsgd_objective(wpsgd_ctx* c, const void* X, wpsgd_xtype xt, int64_t ld_elems, const float* y,
                             int64_t n_rows, const float* w, float lambda, wpsgd_loss loss, double* out) {
  if (!c) return fail(nullptr, WPSGD_ERR_INVALID_ARG, "ctx is NULL");
  if (!w || !out || n_rows < 0 || ld_elems < c->d || (int)loss < 0 || (int)loss > 2 || (n_rows > 0 && (!X || !y)))
    return fail(c, WPSGD_ERR_INVALID_ARG, "objective: bad argument");
  if (xt != WPSGD_X_F32 && xt != WPSGD_X_BF16) return fail(c, WPSGD_ERR_INVALID_ARG, "unknown feature type");
  DeviceGuard guard(c->device);
  const int nblk = grid_for((n_rows + 7) / 8, 1, 148 * 8);
  wpsgd_status s = grow(c, &c->part, &c->part_cap, (size_t)nblk * 2);
  if (s != WPSGD_OK) return s;
  if (xt == WPSGD_X_F32)
    objective_rows_kernel<float><<<nblk, 256, 0, c->stream>>>((const float*)X, ld_elems, y, n_rows, w, c->d, (int)loss, c->part);
  else
    objective_rows_kernel<__nv_bfloat16><<<nblk, 256, 0, c->stream>>>((const __nv_bfloat16*)X, ld_elems, y, n_rows, w, c->d, (int)loss, c->part);
  CU_TRY(c, cudaGetLastError());
  objective_finish_kernel<<<1, 256, 0, c->stream>>>(c->part, nblk, w, c->d, lambda, n_rows, out);
  CU_TRY(c, cudaGetLastError());
  c->launches += 2;
  return WPSGD_OK;
}

wpsgd_status wpsgd_objective_csr(wpsgd_ctx* c, const int64_t* row_ptr, const int32_t* col_idx, const float* val,
                                 const float* y, int64_t n_rows, const float* w, float lambda, wpsgd_loss loss,
                                 double* out) {
  if (!c) return fail(nullptr, WPSGD_ERR_INVALID_ARG, "ctx is NULL");
  if (!w || !out || n_rows < 0 || (int)loss < 0 || (int)loss > 2 || (n_rows > 0 && (!row_ptr || !col_idx || !val || !y)))
    return fail(c, WPSGD_ERR_INVALID_ARG, "objective_csr: bad argument");
  DeviceGuard guard(c->device);
  const int nblk = grid_for((n_rows + 7) / 8, 1, 148 * 8);
  wpsgd_status s = grow(c, &c->part, &c->part_cap, (size_t)nblk * 2);
  if (s != WPSGD_OK) return s;
  objective_rows_csr_kernel<<<nblk, 256, 0, c->stream>>>((const long long*)row_ptr, col_idx, val, y, n_rows, w, (int)loss,
                                                         c->part);
  CU_TRY(c, cudaGetLastError());
  objective_finish_kernel<<<1, 256, 0, c->stream>>>(c->part, nblk, w, c->d, lambda, n_rows, out);
  CU_TRY(c, cudaGetLastError());
  c->launches += 2;
  return WPSGD_OK;
}

wpsgd_status wpsgd_solve_host(wpsgd_ctx* c, const void* X, wpsgd_xtype xt, const float* y, const int64_t* shard_off,
                              const int64_t* n_steps, float eta0, wpsgd_lr sched, float lambda, wpsgd_loss loss,
                              uint64_t seed, const float* w0, double r, float* v_out) {
  if (!c) return fail(nullptr, WPSGD_ERR_INVALID_ARG, "ctx is NULL");
  if (!shard_off || !v_out) return fail(c, WPSGD_ERR_INVALID_ARG, "shard_off or v_out is NULL");
  if (xt != WPSGD_X_F32 && xt != WPSGD_X_BF16) return fail(c, WPSGD_ERR_INVALID_ARG, "unknown feature type");
  DeviceGuard guard(c->device);
  const long long N = shard_off[c->k];
  if (N < 0) return fail(c, WPSGD_ERR_INVALID_ARG, "shard_off[k] < 0");
  if (N > 0 && (!X || !y)) return fail(c, WPSGD_ERR_INVALID_ARG, "X or y is NULL");
  const size_t es = xt == WPSGD_X_F32 ? 4 : 2;
  const size_t xbytes = (size_t)N * (size_t)c->d * es;
  char* sx = (char*)c->st_X;
  wpsgd_status s = grow(c, &sx, &c->st_X_cap, std::max<size_t>(xbytes, 16));
  c->st_X = sx;
  if (s != WPSGD_OK) return s;
  s = grow(c, &c->st_y, &c->st_y_cap, (size_t)std::max(1ll, N));
  if (s != WPSGD_OK) return s;
  if (!c->st_v) CU_TRY(c, cudaMalloc((void**)&c->st_v, (size_t)c->d * sizeof(float)));
  if (w0 && !c->st_w0) CU_TRY(c, cudaMalloc((void**)&c->st_w0, (size_t)c->d * sizeof(float)));
  // Pipelined form: the shards go to the device longest chain first on a copy stream of the context, in up to four
  // groups of nodes, and the chains of a group start as soon as its rows have arrived, so all but the shortest chains
  // run under the remaining copies. Not for rows of at most 64 chunks (their kernel packs nodes into CTAs over the
  // whole node set) and not with fewer than two nodes.
  const long long chunks = c->d / (long long)(16 / es);
  const bool pipelined = c->opt_host_pipeline && N > 0 && c->k >= 2 && n_steps && chunks > 64;
  if (!pipelined) {
    if (N > 0) {
      CU_TRY(c, cudaMemcpyAsync(c->st_X, X, xbytes, cudaMemcpyHostToDevice, c->stream));
      CU_TRY(c, cudaMemcpyAsync(c->st_y, y, (size_t)N * sizeof(float), cudaMemcpyHostToDevice, c->stream));
    }
    if (w0) CU_TRY(c, cudaMemcpyAsync(c->st_w0, w0, (size_t)c->d * sizeof(float), cudaMemcpyHostToDevice, c->stream));
    s = wpsgd_run(c, c->st_X, xt, c->d, c->st_y, shard_off, n_steps, eta0, sched, lambda, loss, seed, w0 ? c->st_w0 : nullptr);
    if (s != WPSGD_OK) return s;
  } else {
    s = check_hyper(c, eta0, (int)sched, lambda, (int)loss);
    if (s != WPSGD_OK) return s;
    for (int j = 0; j < c->k; ++j)
      if (shard_off[j + 1] < shard_off[j] || shard_off[j] < 0) return fail(c, WPSGD_ERR_INVALID_ARG, "shard_off is not non-decreasing");
    if (!c->copy_stream) {
      CU_TRY(c, cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking));
      CU_TRY(c, cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming));
      for (cudaEvent_t& e : c->ev_group) CU_TRY(c, cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
    }
    // the copies start after whatever the caller's stream still does with the staging buffers
    CU_TRY(c, cudaEventRecord(c->ev_fork, c->stream));
    CU_TRY(c, cudaStreamWaitEvent(c->copy_stream, c->ev_fork, 0));
    CU_TRY(c, cudaMemcpyAsync(c->st_y, y, (size_t)N * sizeof(float), cudaMemcpyHostToDevice, c->copy_stream));
    if (w0) CU_TRY(c, cudaMemcpyAsync(c->st_w0, w0, (size_t)c->d * sizeof(float), cudaMemcpyHostToDevice, c->copy_stream));
    std::vector<int> order(c->k);
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return n_steps[a] > n_steps[b]; });  // as make_plan
    const int n_groups = std::min(4, c->k);
    std::vector<LaunchGroup> groups;
    const size_t row_bytes = (size_t)c->d * es;
    int slot = 0;
    for (int g = 0; g < n_groups; ++g) {
      const int count = (c->k - slot + (n_groups - g) - 1) / (n_groups - g);
      for (int q = slot; q < slot + count; ++q) {
        const int j = order[q];
        const size_t off = (size_t)shard_off[j] * row_bytes, len = (size_t)(shard_off[j + 1] - shard_off[j]) * row_bytes;
        if (len > 0)
          CU_TRY(c, cudaMemcpyAsync((char*)c->st_X + off, (const char*)X + off, len, cudaMemcpyHostToDevice, c->copy_stream));
      }
      CU_TRY(c, cudaEventRecord(c->ev_group[g], c->copy_stream));
      groups.push_back({count, c->ev_group[g]});
      slot += count;
    }
    c->eta0 = eta0; c->sched = (int)sched; c->lambda = lambda; c->loss = (int)loss; c->seed = seed;
    c->have_run = false;
    s = run_dense_common(c, c->st_X, xt, c->d, c->st_y, (const long long*)shard_off, (const long long*)n_steps,
                         w0 ? c->st_w0 : nullptr, false, &groups);
    if (s != WPSGD_OK) return s;
  }
  s = wpsgd_combine(c, r, c->st_v);
  if (s != WPSGD_OK) return s;
  CU_TRY(c, cudaMemcpyAsync(v_out, c->st_v, (size_t)c->d * sizeof(float), cudaMemcpyDeviceToHost, c->stream));
  CU_TRY(c, cudaStreamSynchronize(c->stream));
  return WPSGD_OK;
}

wpsgd_status wpsgd_solve_host_csr(wpsgd_ctx* c, const int64_t* row_ptr, const int32_t* col_idx, const float* val, const float* y,
                                  const int64_t* shard_off, const int64_t* n_steps, float eta0, wpsgd_lr sched, float lambda,
                                  wpsgd_loss loss, uint64_t seed, const float* w0, double r, float* v_out) {
  if (!c) return fail(nullptr, WPSGD_ERR_INVALID_ARG, "ctx is NULL");
  if (!shard_off || !v_out) return fail(c, WPSGD_ERR_INVALID_ARG, "shard_off or v_out is NULL");
  DeviceGuard guard(c->device);
  const long long N = shard_off[c->k];
  if (N < 0) return fail(c, WPSGD_ERR_INVALID_ARG, "shard_off[k] < 0");
  if (N > 0 && (!row_ptr || !y)) return fail(c, WPSGD_ERR_INVALID_ARG, "row_ptr or y is NULL");
  const long long nnz = N > 0 ? row_ptr[N] : 0;
  if (nnz < 0 || (nnz > 0 && (!col_idx || !val))) return fail(c, WPSGD_ERR_INVALID_ARG, "row_ptr[N] < 0, or col_idx / val is NULL");
  wpsgd_status s = grow(c, &c->st_rp, &c->st_rp_cap, (size_t)N + 1);
  if (s != WPSGD_OK) return s;
  s = grow(c, &c->st_ci, &c->st_ci_cap, (size_t)std::max(1ll, nnz));
  if (s != WPSGD_OK) return s;
  s = grow(c, &c->st_va, &c->st_va_cap, (size_t)std::max(1ll, nnz));
  if (s != WPSGD_OK) return s;
  s = grow(c, &c->st_y, &c->st_y_cap, (size_t)std::max(1ll, N));
  if (s != WPSGD_OK) return s;
  if (!c->st_v) CU_TRY(c, cudaMalloc((void**)&c->st_v, (size_t)c->d * sizeof(float)));
  if (w0 && !c->st_w0) CU_TRY(c, cudaMalloc((void**)&c->st_w0, (size_t)c->d * sizeof(float)));
  if (N > 0) {
    CU_TRY(c, cudaMemcpyAsync(c->st_rp, row_ptr, ((size_t)N + 1) * sizeof(long long), cudaMemcpyHostToDevice, c->stream));
    CU_TRY(c, cudaMemcpyAsync(c->st_y, y, (size_t)N * sizeof(float), cudaMemcpyHostToDevice, c->stream));
  }
  if (nnz > 0) {
    CU_TRY(c, cudaMemcpyAsync(c->st_ci, col_idx, (size_t)nnz * sizeof(int), cudaMemcpyHostToDevice, c->stream));
    CU_TRY(c, cudaMemcpyAsync(c->st_va, val, (size_t)nnz * sizeof(float), cudaMemcpyHostToDevice, c->stream));
  }
  if (w0) CU_TRY(c, cudaMemcpyAsync(c->st_w0, w0, (size_t)c->d * sizeof(float), cudaMemcpyHostToDevice, c->stream));
  s = wpsgd_run_csr(c, (const int64_t*)c->st_rp, c->st_ci, c->st_va, c->st_y, shard_off, n_steps, eta0, sched, lambda, loss, seed,
                    w0 ? c->st_w0 : nullptr);
  if (s != WPSGD_OK) return s;
  s = wpsgd_combine(c, r, c->st_v);
  if (s != WPSGD_OK) return s;
  CU_TRY(c, cudaMemcpyAsync(v_out, c->st_v, (size_t)c->d * sizeof(float), cudaMemcpyDeviceToHost, c->stream));
  CU_TRY(c, cudaStreamSynchronize(c->stream));
  return WPSGD_OK;
}

wpsgd_status wpsgd_solve_static(int device, void* cuda_stream, const void* X, wpsgd_xtype xt, int64_t ld_elems,
                                const float* y, const int64_t* shard_off, const int64_t* n_steps, int32_t k, int64_t d,
                                float eta0, wpsgd_lr sched, float lambda, wpsgd_loss loss, uint64_t seed,
                                const float* w0, double r, float* v_out) {
  if (k < 1 || d < 1) return fail(nullptr, WPSGD_ERR_INVALID_ARG, "solve_static: k and d must be >= 1");
  if (!shard_off || !n_steps || !v_out) return fail(nullptr, WPSGD_ERR_INVALID_ARG, "solve_static: shard_off, n_steps or v_out is NULL");
  char msg[200];
  if (k > WPSGD_STATIC_MAX_NODES) {
    snprintf(msg, sizeof(msg), "solve_static: k = %d exceeds the built-in maximum of %d nodes", (int)k, WPSGD_STATIC_MAX_NODES);
    return fail(nullptr, WPSGD_ERR_UNSUPPORTED, msg);
  }
  if ((long long)k * (long long)d > WPSGD_STATIC_MAX_MODEL_ELEMS) {
    snprintf(msg, sizeof(msg), "solve_static: k * d = %lld exceeds the built-in maximum of %lld model elements",
             (long long)k * (long long)d, (long long)WPSGD_STATIC_MAX_MODEL_ELEMS);
    return fail(nullptr, WPSGD_ERR_UNSUPPORTED, msg);
  }
  long long total = 0;
  for (int j = 0; j < k; ++j) {
    if (n_steps[j] < 0) return fail(nullptr, WPSGD_ERR_INVALID_ARG, "solve_static: negative step count");
    total += n_steps[j];
    if (total > WPSGD_STATIC_MAX_STEPS) {
      snprintf(msg, sizeof(msg), "solve_static: the step counts add up to more than the built-in maximum of %lld",
               (long long)WPSGD_STATIC_MAX_STEPS);
      return fail(nullptr, WPSGD_ERR_UNSUPPORTED, msg);
    }
  }
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) {
    cudaGetLastError();
    return fail(nullptr, WPSGD_ERR_CUDA, "no CUDA device available");
  }
  if (device < 0 || device >= ndev || device >= kStaticMaxDevices)
    return fail(nullptr, WPSGD_ERR_INVALID_ARG, "solve_static: device index out of range");
  DeviceGuard guard(device);
  unsigned char* base = nullptr;
  wpsgd_status s = static_scratch_base(device, &base);
  if (s != WPSGD_OK) return s;

  // A context on the host stack whose device pointers all lie inside the built-in array. It is never
  // handed to wpsgd_destroy: nothing in it was allocated, so nothing is freed.
  wpsgd_ctx c;
  c.device = device;
  c.stream = (cudaStream_t)cuda_stream;
  c.k = k;
  c.d = d;
  c.steps_done.assign(k, 0);
  c.node_ids.resize(k);
  std::iota(c.node_ids.begin(), c.node_ids.end(), 0);
  const StaticLayout L;
  c.W = (float*)(base + L.W);
  c.idx = (uint32_t*)(base + L.idx);
  c.idx_cap = (size_t)WPSGD_STATIC_MAX_STEPS + 64 * WPSGD_STATIC_MAX_NODES;  // never regrown: padding included
  c.t_shard_off = (long long*)(base + L.shard_off);
  c.t_steps = (long long*)(base + L.steps);
  c.t_first = (long long*)(base + L.first);
  c.t_idx_off = (long long*)(base + L.idx_off);
  c.t_rows = (long long*)(base + L.rows);
  c.t_count = (long long*)(base + L.count);
  c.t_order = (int*)(base + L.order);
  c.t_ids = (int*)(base + L.ids);
  c.t_group = (int*)(base + L.group);
  c.t_weights = (double*)(base + L.weights);
  c.scale = (double*)(base + L.scale);
  c.status = (DevStatus*)(base + L.status);
  // the array keeps what the previous call left: the status word is the one thing that must start at zero
  // (models, tables and the sample stream are fully rewritten for the sizes of this call)
  cudaError_t e = cudaMemsetAsync(c.status, 0, sizeof(DevStatus), c.stream);
  if (e != cudaSuccess) return fail(nullptr, WPSGD_ERR_CUDA, std::string("solve_static: cudaMemsetAsync: ") + cudaGetErrorString(e));
  s = wpsgd_run(&c, X, xt, ld_elems, y, shard_off, n_steps, eta0, sched, lambda, loss, seed, w0);
  if (s == WPSGD_OK) s = wpsgd_combine(&c, r, v_out);
  if (s != WPSGD_OK) g_err = "solve_static: " + c.err;
  return s;
}

wpsgd_status wpsgd_check(wpsgd_ctx* c) {
  if (!c) return fail(nullptr, WPSGD_ERR_INVALID_ARG, "ctx is NULL");
  DeviceGuard guard(c->device);
  return read_status(c, c->status, c->stream);
}

wpsgd_status wpsgd_check_static(int device, void* cuda_stream) {
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) {
    cudaGetLastError();
    return fail(nullptr, WPSGD_ERR_CUDA, "no CUDA device available");
  }
  if (device < 0 || device >= ndev || device >= kStaticMaxDevices)
    return fail(nullptr, WPSGD_ERR_INVALID_ARG, "check_static: device index out of range");
  DeviceGuard guard(device);
  unsigned char* base = nullptr;
  wpsgd_status s = static_scratch_base(device, &base);
  if (s != WPSGD_OK) return s;
  return read_status(nullptr, (DevStatus*)(base + StaticLayout().status), (cudaStream_t)cuda_stream);
}

int64_t wpsgd_launch_count(const wpsgd_ctx* c) { return c ? c->launches : 0; }

const char* wpsgd_last_error(const wpsgd_ctx* c) { return c ? c->err.c_str() : g_err.c_str(); }

}  // extern "C"
