// Shared device-side helpers of the WP-SGD kernels: status word, loss derivatives, step size,
// small reductions. Everything here is used by the CUDA path only.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace wpsgd {

// Device status word, owned by the context. code != 0 after a kernel detected a problem.
struct DevStatus {
  int code;   // 0 ok, 1 bounded wait gave up, 2 bounds check failed
  int where;  // kernel-specific location tag
  long long detail;
};
enum { DEV_OK = 0, DEV_TIMEOUT = 1, DEV_BOUNDS = 2 };

__device__ __forceinline__ void set_status(DevStatus* st, int code, int where, long long detail) {
  if (atomicCAS(&st->code, 0, code) == 0) {
    st->where = where;
    st->detail = detail;
  }
}

enum { LOSS_HINGE = 0, LOSS_LOGISTIC = 1, LOSS_SQUARED = 2 };
enum { LR_CONST = 0, LR_INV_SQRT = 1 };

// dL/dz of the three losses at (y, z) (Eq. 4: L is a convex function of the margin z = w.x).
__device__ __forceinline__ float loss_derivative(int loss, float y, float z) {
  if (loss == LOSS_HINGE) return (y * z < 1.0f) ? -y : 0.0f;
  if (loss == LOSS_LOGISTIC) return -y / (1.0f + expf(y * z));
  return z - y;
}

// eta_n for the 1-based step number n.
__device__ __forceinline__ float step_size(float eta0, int sched, long long n) {
  return sched == LR_INV_SQRT ? eta0 / sqrtf((float)n) : eta0;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// 16-byte vector of features, widened to fp32. V = elements per 16 bytes.
template <typename XT>
struct XVec;
template <>
struct XVec<float> {
  static constexpr int V = 4;
  __device__ __forceinline__ static void widen(const uint4& raw, float (&f)[4]) {
    f[0] = __uint_as_float(raw.x);
    f[1] = __uint_as_float(raw.y);
    f[2] = __uint_as_float(raw.z);
    f[3] = __uint_as_float(raw.w);
  }
};
template <>
struct XVec<__nv_bfloat16> {
  static constexpr int V = 8;
  // bf16 -> fp32 is a 16-bit left shift of the bit pattern (exact).
  __device__ __forceinline__ static void widen(const uint4& raw, float (&f)[8]) {
    f[0] = __uint_as_float(raw.x << 16);
    f[1] = __uint_as_float(raw.x & 0xffff0000u);
    f[2] = __uint_as_float(raw.y << 16);
    f[3] = __uint_as_float(raw.y & 0xffff0000u);
    f[4] = __uint_as_float(raw.z << 16);
    f[5] = __uint_as_float(raw.z & 0xffff0000u);
    f[6] = __uint_as_float(raw.w << 16);
    f[7] = __uint_as_float(raw.w & 0xffff0000u);
  }
};

template <typename XT>
__device__ __forceinline__ float widen_scalar(XT v);
template <>
__device__ __forceinline__ float widen_scalar<float>(float v) { return v; }
template <>
__device__ __forceinline__ float widen_scalar<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

// Read-only 16-byte global load that does not allocate in L1 (rows are streamed once per visit).
__device__ __forceinline__ uint4 ld_stream16(const void* p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p));
  return r;
}

}  // namespace wpsgd
