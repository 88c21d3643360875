// Declarations shared by the preprocessing kernels.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp4.h>
#include <cuda_fp8.h>

#include "vc_internal.h"
#include "vc_sm100.cuh"

namespace vc {

using namespace sm100;

struct RopeDesc {
  int pair_start[3];   // first channel pair of each axis
  int pairs[3];        // channel pairs per axis
  int off[3];          // entry offset of each axis table
  int len[3];          // positions per axis
  int entries;
  int grid_h, grid_w;
  unsigned long long mul_w, mul_h;   // ceil(2^40 / divisor)
};

struct PrepArgs {
  const __nv_bfloat16 *q, *k, *v;
  const int32_t* perm;
  int64_t stride_b, stride_h, stride_n;
  int stride_n_bytes;               // 2 * stride_n (a row stride fits 32 bits: checked when the call is resolved)
  unsigned long long mul_H;         // ceil(2^40 / H): bh / H by one multiplication
  int H, N, n_pad, nb, bh0, flags, rope_in_smem, rope_default;
  uint8_t *q_codes, *k_codes, *v_codes, *q_micro, *k_micro, *v_micro;
  float *q_scale, *k_scale, *v_scale, *k_mean;
  __nv_bfloat16* v_means;
  const float2* rope;
  float *k_part, *v_mu;
  unsigned int *v_amax, *qk_amax;   // qk_amax: [2][BH]
  const float* ext_k_mean;          // caller-supplied statistics (vc_prep_with_stats), else null
  int BH;
  RopeDesc rd;
};

__device__ __forceinline__ unsigned int div40(unsigned int x, unsigned long long mul) {
  return (unsigned int)(((unsigned long long)x * mul) >> 40);
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, s));
  return v;
}

__device__ __forceinline__ float e4m3_to_float(unsigned int code) {
  __half_raw h = __nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)code, __NV_E4M3);
  return __half2float(__half(h));
}

__device__ __forceinline__ void cp_async16(void* dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Token position -> (t, y, x) of the grid.
__device__ __forceinline__ void grid_pos(const RopeDesc& rd, int src, int& tt, int& ty, int& tx) {
  const unsigned int q1 = div40((unsigned)src, rd.mul_w);
  tx = src - q1 * rd.grid_w;
  tt = div40(q1, rd.mul_h);
  ty = q1 - tt * rd.grid_h;
}


}  // namespace vc
