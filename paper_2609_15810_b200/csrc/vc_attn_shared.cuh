// Pieces shared by the 8-bit and 4-bit attention kernels: the barrier block of the
// two-query-tile pipeline, bounded waits, the block-mean operand layout, TMA descriptors.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "vc_internal.h"
#include "vc_sm100.cuh"

namespace vc {
namespace attn {

using namespace sm100;

constexpr uint32_t kErrTimeout = kStatusTimeout;

// Arguments of the 8-bit attention kernels.
struct AttnArgs {
  const float *q_scale, *k_scale, *v_scale;
  const __nv_bfloat16* v_means;
  __nv_bfloat16* o;
  uint32_t* status;
  int N, n_pad, nb, p_format;
  float sl;        // softmax_scale * log2(e)
  float code_off;  // 120 + beta  (Eq. 7)
  uint32_t wait_limit;   // polls after which a wait gives up
  uint32_t wait_hint_ns;
};

constexpr int kStages2 = 4;
constexpr uint32_t kWaitLimit2 = 1u << 18;   // default polls of a wait, x up to 4 us per try: about one second
constexpr uint32_t kDrainLimit = 1u << 22;   // polls of the exit waits for a CTA's own copies and MMAs

inline uint32_t attn_wait_limit() {
  const uint32_t lim = wait_limit_override();
  return lim ? lim : kWaitLimit2;
}
// with the test override a poll never sleeps (hint 0 selects non-blocking tests of the barrier),
// so that a tiny limit really is a short wait
inline uint32_t attn_wait_hint_ns() { return wait_limit_override() ? 0u : 4000u; }

struct FaSmem {
  uint64_t q_full, kv_full[kStages2], kv_empty[kStages2];
  uint64_t s_full[2], s_free[2], o_done[2], fin_full[2], o_final[2];
  // alpha and codes+correction hand-offs can run one key tile ahead of their consumer, so they
  // alternate between two barriers (a parity wait aliases after two phases)
  uint64_t a_full[2][2], pc_full[2][2];
  uint64_t drain[2];      // exit: "every MMA this issuer warp issued has completed"
  float alpha[2][128];
  uint32_t tmem_base;
  uint32_t wait_limit;    // polls of a wait ...
  uint32_t wait_hint_ns;  // ... each of which may sleep this long in hardware
  volatile int abort;
};

__device__ __forceinline__ bool wait2(uint64_t* bar, uint32_t parity, FaSmem* sh, uint32_t* status, uint32_t code) {
  const uint32_t limit = sh->wait_limit, hint = sh->wait_hint_ns;
  if (hint) {
    if (mbar_try_wait(bar, parity)) return true;
    for (uint32_t i = 0; i < limit; ++i) {
      if (mbar_try_wait_hint(bar, parity, hint)) return true;
      if ((i & 63u) == 63u && sh->abort) return false;
    }
  } else {                                     // test hook: polls that never sleep
    for (uint32_t i = 0; i < limit; ++i) {
      if (mbar_test_wait(bar, parity)) return true;
      if ((i & 63u) == 63u && sh->abort) return false;
    }
  }
  sh->abort = 1;
  atomicExch(status, kErrTimeout | code);
  return false;
}
__device__ __forceinline__ bool warp_wait2(uint64_t* bar, uint32_t parity, FaSmem* sh, uint32_t* status, uint32_t code) {
  return __all_sync(0xffffffffu, wait2(bar, parity, sh, status, code));
}

// Exit protocol of the pipelined kernels.  A CTA may leave early (a wait gave up and set `abort`),
// and even then nothing it started may outlive it: shared memory and tensor memory go back to
// the SM when the CTA exits, so a bulk copy still landing or an MMA still reading would touch
// memory that belongs to somebody else by then.
//   producer warp   waits (bounded, generous) for every copy it issued and nobody consumed
//   issuer warps    commit to their own barrier and wait for it: all their MMAs have completed
// tcgen05.ld / tcgen05.st of the other warps are complete at their wait::ld / wait::st.  Only
// then does the CTA reach the barrier in front of the tensor-memory release.
__device__ __forceinline__ void drain_loads(FaSmem* sh, int issued) {
  mbar_wait(&sh->q_full, 0, kDrainLimit);
  for (int jj = issued > kStages2 ? issued - kStages2 : 0; jj < issued; ++jj)
    mbar_wait(&sh->kv_full[jj % kStages2], (jj / kStages2) & 1, kDrainLimit);
}
__device__ __forceinline__ void drain_mmas(FaSmem* sh, int which) {
  if (elect_one()) mma_commit(&sh->drain[which]);
  __syncwarp();
  mbar_wait(&sh->drain[which], 0, kDrainLimit);
}

// Block means as the B operand of the per-tile mean-restoration MMA: per (b, h, key tile) a
// [d][8] fp32 tile with entry [c][0] = [c][1] = mu~[c] (for r_hi and r_lo) and zeros elsewhere.
template <int D>
__global__ void means_tile_layout_kernel(const __nv_bfloat16* __restrict__ means, float* __restrict__ out, size_t n) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;   // (bh * nb + tile) * D + c
  if (i >= n) return;
  const float v = __bfloat162float(means[i]);
  float4* dst = reinterpret_cast<float4*>(out + i * 8);
  dst[0] = make_float4(v, v, 0.f, 0.f);
  dst[1] = make_float4(0.f, 0.f, 0.f, 0.f);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;   // resolved once; the driver entry point never changes
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// 3-D byte tensor [dim2][dim1][dim0], box {box0, box1, 1}, swizzle chosen by the box width.
inline bool make_map(CUtensorMap* m, const void* base, uint64_t dim0, uint64_t dim1, uint64_t dim2, uint32_t box0, uint32_t box1) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[3] = {dim0, dim1, dim2};
  const cuuint64_t strides[2] = {dim0, dim0 * dim1};
  const cuuint32_t box[3] = {box0, box1, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUtensorMapSwizzle sw = box0 == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : (box0 == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}


// 3-D tensor of packed 4-bit elements [dim2][dim1][dim0 elements]; a box of 128 elements x box1
// rows lands in shared memory as 128-byte rows of 16-byte containers (16 elements in the low 8
// bytes, 128-byte swizzle): the layout kind::mxf8f6f4 reads 4-bit operands in.  The copy reports
// the packed bytes (64 per row) to its mbarrier.  `base` must be 32-byte aligned, dim0 a
// multiple of 128.
inline bool make_map_u4(CUtensorMap* m, const void* base, uint64_t dim0, uint64_t dim1, uint64_t dim2, uint32_t box1) {
  EncodeTiledFn fn = encode_fn();
  if (!fn || ((uintptr_t)base & 31) || (dim0 & 127)) return false;
  const cuuint64_t dims[3] = {dim0, dim1, dim2};
  const cuuint64_t strides[2] = {dim0 / 2, dim0 / 2 * dim1};
  const cuuint32_t box[3] = {128, box1, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_16U4_ALIGN16B, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace attn
}  // namespace vc
