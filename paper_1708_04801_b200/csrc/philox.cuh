// Sample-index stream of the chains: Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11), written
// from the published definition, and the kernel that materialises each node's stream.
//
// Stands for Algorithm 1's "randomly shuffle the data on machine i; get the n-th example": the
// n-th example (1-based) of node j is row floor(u * m_j / 2^32) of its shard, u being output word
// (n-1)&3 of the block with counter ((n-1)>>2 low, (n-1)>>2 high, j, 0) and key (seed low, seed high).
#pragma once

#include "common.cuh"

namespace wpsgd {

// High 32 bits of a 32 x 32 -> 64 bit product, on the device and on the host.
__host__ __device__ __forceinline__ uint32_t mulhi32(uint32_t a, uint32_t b) {
#ifdef __CUDA_ARCH__
  return __umulhi(a, b);
#else
  return (uint32_t)(((unsigned long long)a * (unsigned long long)b) >> 32);
#endif
}

__host__ __device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int i = 0; i < 10; ++i) {
    const uint32_t hi0 = mulhi32(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
    const uint32_t hi1 = mulhi32(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
    c = make_uint4(hi1 ^ c.y ^ k0, lo1, hi0 ^ c.w ^ k1, lo0);
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return c;
}

// ---- shuffled order: one keyed permutation of the shard per node, cycled (Algorithm 1 read literally: "randomly
// shuffle the data on machine i", then "get the n-th example") -------------------------------------------------
// The n-th example is row pi((n-1) mod m). pi is a 4-round balanced Feistel network on 2w bits (2w = the even
// bit count >= 2 covering m-1) with cycle walking; round keys = the Philox block at counter (0, 0, node, 1);
// round function = a 32-bit multiply / xor-shift mixer masked to w bits.
__host__ __device__ __forceinline__ uint32_t mix_round(uint32_t x, uint32_t key) {
  uint32_t h = x ^ key;
  h *= 0x85EBCA6Bu;
  h ^= h >> 13;
  h *= 0xC2B2AE35u;
  h ^= h >> 16;
  return h;
}

__host__ __device__ __forceinline__ uint32_t shuffled_row(const uint4& keys, long long step0 /*0-based*/, uint32_t m) {
  if (m <= 1u) return 0u;
  int bits = 0;  // smallest bits with 2^bits >= m (m >= 2)
  while (bits < 32 && ((m - 1u) >> bits) != 0u) ++bits;
  if (bits < 2) bits = 2;
  if (bits & 1) ++bits;
  const int w = bits >> 1;
  const uint32_t mask = (w == 16) ? 0xFFFFu : ((1u << w) - 1u);
  const uint32_t kk[4] = {keys.x, keys.y, keys.z, keys.w};
  unsigned long long x = (unsigned long long)(step0 % (long long)m);
  // Every pass is a bijection of [0, 2^bits), so walking from a value below m returns below m; 2^bits < 4m, and
  // the expected number of passes is below 4. The loop bound only guards against a broken invariant.
  for (int guard = 0; guard < (1 << 20); ++guard) {
    uint32_t L = (uint32_t)(x >> w), R = (uint32_t)x & mask;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint32_t t = (L ^ mix_round(R, kk[i])) & mask;
      L = R;
      R = t;
    }
    x = ((unsigned long long)L << w) | R;
    if (x < m) break;
  }
  return (uint32_t)(x < m ? x : 0ull);
}

// Entries of steps b+1 .. b+cnt of node j (shard of m rows) into out[0 .. cnt). sampling 0: one counter value q
// (four consecutive steps) per (t0 + i * stride); sampling 1: one step per (t0 + i * stride).
__host__ __device__ __forceinline__ void emit_indices(int sampling, uint64_t seed, uint32_t j, long long b, long long cnt, uint32_t m,
                                             uint32_t* __restrict__ out, long long t0, long long stride) {
  if (sampling == 1) {
    const uint4 keys = philox4x32_10(make_uint4(0u, 0u, j, 1u), (uint32_t)seed, (uint32_t)(seed >> 32));
    for (long long i = t0; i < cnt; i += stride) out[i] = shuffled_row(keys, b + i, m);
    return;
  }
  const long long q_lo = b >> 2, q_hi = (b + cnt - 1) >> 2;  // zero-based step s = n-1 lies in [b, b+cnt)
  for (long long q = q_lo + t0; q <= q_hi; q += stride) {
    const uint4 o = philox4x32_10(make_uint4((uint32_t)q, (uint32_t)((unsigned long long)q >> 32), j, 0u),
                                  (uint32_t)seed, (uint32_t)(seed >> 32));
    const uint32_t w[4] = {o.x, o.y, o.z, o.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const long long s = (q << 2) + e;
      if (s >= b && s < b + cnt) out[s - b] = mulhi32(w[e], m);  // floor(u m / 2^32)
    }
  }
}

// All nodes' streams for one launch of the chains. Node = blockIdx.y (+ gridDim.y per pass).
//   idx_off[j]   position of node j's first entry in idx (prefix sums of count)
//   first[j]     number of steps node j has already run (its entries start at step first[j]+1)
//   count[j]     entries to produce for node j
//   rows[j]      shard size m_j
//   ids[j]       node number that enters the counter (j itself unless the caller renumbers nodes)
__global__ void index_stream_kernel(int sampling, uint64_t seed, int k, const long long* __restrict__ idx_off,
                                    const long long* __restrict__ first, const long long* __restrict__ count,
                                    const long long* __restrict__ rows, const int* __restrict__ ids,
                                    uint32_t* __restrict__ idx) {
  for (int j = blockIdx.y; j < k; j += gridDim.y) {
    const long long cnt = count[j];
    if (cnt <= 0) continue;
    emit_indices(sampling, seed, (uint32_t)ids[j], first[j], cnt, (uint32_t)rows[j], idx + idx_off[j],
                 (long long)blockIdx.x * blockDim.x + threadIdx.x, (long long)gridDim.x * blockDim.x);
  }
}

// One node's stream, for callers that want to look at it.
__global__ void index_single_kernel(int sampling, uint64_t seed, int node, long long m, long long n_begin,
                                    long long count, uint32_t* __restrict__ out) {
  if (count > 0)
    emit_indices(sampling, seed, (uint32_t)node, n_begin, count, (uint32_t)m, out,
                 (long long)blockIdx.x * blockDim.x + threadIdx.x, (long long)gridDim.x * blockDim.x);
}

}  // namespace wpsgd
