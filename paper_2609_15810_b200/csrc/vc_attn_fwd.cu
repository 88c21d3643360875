// Quantized attention forward of VC-Attention for sm_100a (Eq. 1, Eq. 6, Eq. 7).
//
// One CTA owns one 128-row query tile of one (batch, head) and streams the permuted
// key/value tiles of 128 tokens through it:
//   TMA (cp.async.bulk.tensor, 128-byte swizzle)  K^_j, R^_j  -> shared memory
//   tcgen05.mma kind::f8f6f4 (E4M3 x E4M3, FP32)  S = Q^ K^_j^T -> tensor memory
//   softmax stage, one thread per query row        running max, alpha, ExpCast-FP8 code
//                                                  (one FMA + round, no exponential)
//   P^ codes -> tensor memory (A operand)          tcgen05.st
//   tcgen05.mma                                    A += P^ R^_j
//   mean restoration                               A = alpha A + r mu~_j  (Eq. 6)
// Epilogue: O = s_V * A / l, bf16, original query order.
#include <cuda_bf16.h>
#include <cuda_fp8.h>

#include "vc_internal.h"
#include "vc_sm100.cuh"

namespace vc {
namespace {

using namespace sm100;

constexpr uint32_t kErrTimeout = 0x100;

struct AttnArgs {
  const float *q_scale, *k_scale, *v_scale;
  const __nv_bfloat16* v_means;
  __nv_bfloat16* o;
  uint32_t* status;
  int N, n_pad, nb, p_format;
  float sl;        // softmax_scale * log2(e)
  float code_off;  // 120 + beta  (Eq. 7)
};

// Value of an ExpCast / E4M3 code in [0, 126] (non-negative): normals by placing the
// exponent and mantissa fields into an fp32 pattern, subnormals (codes 1..7) as m * 2^-9.
__device__ __forceinline__ float decode_pos_e4m3(uint32_t code) {
  return code >= 8u ? __uint_as_float((code + 960u) << 20) : (float)code * 0.001953125f;
}

template <int D>
__global__ void __launch_bounds__(128)
attn_fwd_serial_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                       const __grid_constant__ CUtensorMap tm_v, const AttnArgs a) {
  constexpr int kTmemCols = 256;
  constexpr uint32_t S_COL = 0, O_COL = 128;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char* sQ = smem;                         // 128 rows x D bytes
  unsigned char* sK = smem + 128 * D;               // 128 rows x D bytes
  unsigned char* sV = smem + 2 * 128 * D;           // D rows x 128 bytes
  float* sMu = reinterpret_cast<float*>(smem + 2 * 128 * D + D * 128);
  uint64_t* bars = reinterpret_cast<uint64_t*>(sMu + D);
  uint64_t *bar_q = bars, *bar_kv = bars + 1, *bar_s = bars + 2, *bar_o = bars + 3;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 4);

  const int tid = threadIdx.x, warp = tid >> 5;
  const int qblk = blockIdx.x, bh = blockIdx.y;
  bool alive = true;   // false after a timed-out wait: skip all further waits

  if (tid == 0) {
    mbar_init(bar_q, 1); mbar_init(bar_kv, 1); mbar_init(bar_s, 1); mbar_init(bar_o, 1);
    mbar_fence_init();
    tma_prefetch_desc(&tm_q); tma_prefetch_desc(&tm_k); tma_prefetch_desc(&tm_v);
  }
  if (warp == 0) { tmem_alloc<kTmemCols>(tmem_slot); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);

  if (tid == 0) {
    mbar_expect_tx(bar_q, 128 * D);
    tma_load_3d(sQ, &tm_q, bar_q, 0, qblk * 128, bh);
  }
  if (!mbar_wait(bar_q, 0)) { alive = false; atomicExch(a.status, kErrTimeout | 1); }

  const float sq = a.q_scale[(size_t)bh * a.nb + qblk];
  const uint32_t idesc_qk = idesc_e4m3(128, 128);
  const uint32_t idesc_pv = idesc_e4m3(128, D);
  const uint64_t dq = smem_desc_kmajor(smem_u32(sQ), D);
  const uint64_t dk = smem_desc_kmajor(smem_u32(sK), D);
  const uint64_t dv = smem_desc_kmajor(smem_u32(sV), 128);

  float m_run = -INFINITY, l_run = 0.f;
  for (int j = 0; j < a.nb; ++j) {
    const uint32_t ph = j & 1;
    if (tid == 0) {
      mbar_expect_tx(bar_kv, 2 * 128 * D);
      tma_load_3d(sK, &tm_k, bar_kv, 0, j * 128, bh);
      tma_load_3d(sV, &tm_v, bar_kv, j * 128, 0, bh);
    }
    if (tid < D / 2) {
      const __nv_bfloat162 m2 = *reinterpret_cast<const __nv_bfloat162*>(a.v_means + ((size_t)bh * a.nb + j) * D + 2 * tid);
      sMu[2 * tid] = __low2float(m2);
      sMu[2 * tid + 1] = __high2float(m2);
    }
    const float cs = (sq * a.k_scale[(size_t)bh * a.nb + j]) * a.sl;   // code units -> log2 domain
    if (alive && !mbar_wait(bar_kv, ph)) { alive = false; atomicExch(a.status, kErrTimeout | 2); }
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
#pragma unroll
      for (int k = 0; k < D / 32; ++k) mma_f8_ss(tmem + S_COL, dq + 2 * k, dk + 2 * k, idesc_qk, k > 0);
      mma_commit(bar_s);
    }
    if (alive && !mbar_wait(bar_s, ph)) { alive = false; atomicExch(a.status, kErrTimeout | 3); }
    tc_fence_after();

    // ---- softmax stage: this thread owns query row 32*warp + lane
    const int nv = min(128, a.N - j * 128);   // valid keys in this tile
    uint32_t r[32];
    float mx = -INFINITY;
#pragma unroll 1
    for (int c = 0; c < 4; ++c) {
      tmem_ld32(lane_base + S_COL + 32 * c, r);
      tmem_wait_ld();
#pragma unroll
      for (int i = 0; i < 32; ++i)
        if (32 * c + i < nv) mx = fmaxf(mx, __uint_as_float(r[i]));
    }
    const float m_new = fmaxf(m_run, mx * cs);                 // m' = max(m, rowmax S_ij)
    const float alpha = exp2f(m_run - m_new);                  // 0 on the first tile
    float rsum = 0.f;
#pragma unroll 1
    for (int c = 0; c < 4; ++c) {
      tmem_ld32(lane_base + S_COL + 32 * c, r);
      tmem_wait_ld();
      uint32_t pk[8];
#pragma unroll
      for (int w = 0; w < 8; ++w) {
        uint32_t word = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int i = 4 * w + e;
          const float s = __uint_as_float(r[i]);
          uint32_t code;
          if (a.p_format == VC_P_EXPCAST_E4M3) {
            // Eq. 7: c = 8 u + (120 + beta), clipped to [0, 120], rounded to nearest even
            const float u = fmaf(s, cs, -m_new);
            const float t = fminf(fmaxf(fmaf(u, 8.0f, a.code_off), 0.0f), 120.0f);
            code = (uint32_t)__float2int_rn(t);
          } else {
            const float u = fmaf(s, cs, -m_new);
            code = (uint32_t)__nv_cvt_float_to_fp8(exp2f(u + 8.0f), __NV_SATFINITE, __NV_E4M3);
          }
          if (32 * c + i >= nv) code = 0;                      // padded keys carry code 0
          rsum += decode_pos_e4m3(code);
          word |= code << (8 * e);
        }
        pk[w] = word;
      }
      tmem_st8(lane_base + S_COL + 8 * c, pk);                 // P^ aliases the consumed part of S
    }
    l_run = alpha * l_run + rsum;                              // l <- alpha l + r
    m_run = m_new;

    // ---- A <- alpha A + r mu~_j  (Eq. 6); the P^ R^ product is added by the MMA below
#pragma unroll 1
    for (int c = 0; c < D / 32; ++c) {
      if (j > 0) { tmem_ld32(lane_base + O_COL + 32 * c, r); tmem_wait_ld(); }
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        const float prev = j > 0 ? __uint_as_float(r[i]) * alpha : 0.f;
        r[i] = __float_as_uint(fmaf(rsum, sMu[32 * c + i], prev));
      }
      tmem_st32(lane_base + O_COL + 32 * c, r);
    }
    tmem_wait_st();
    tc_fence_before();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
#pragma unroll
      for (int k = 0; k < 4; ++k) mma_f8_ts(tmem + O_COL, tmem + S_COL + 8 * k, dv + 2 * k, idesc_pv, 1);
      mma_commit(bar_o);
    }
    if (alive && !mbar_wait(bar_o, ph)) { alive = false; atomicExch(a.status, kErrTimeout | 4); }
    tc_fence_after();
  }

  // ---- epilogue: O = s_V * A / l
  const int row = qblk * 128 + tid;
  const float inv_l = 1.0f / l_run;
  uint32_t r[32];
#pragma unroll 1
  for (int c = 0; c < D / 32; ++c) {
    tmem_ld32(lane_base + O_COL + 32 * c, r);
    tmem_wait_ld();
    if (row < a.N) {
      uint32_t out[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const float x0 = __uint_as_float(r[2 * i]) * inv_l * a.v_scale[(size_t)bh * D + 32 * c + 2 * i];
        const float x1 = __uint_as_float(r[2 * i + 1]) * inv_l * a.v_scale[(size_t)bh * D + 32 * c + 2 * i + 1];
        __nv_bfloat162 h2 = __floats2bfloat162_rn(x0, x1);
        out[i] = *reinterpret_cast<uint32_t*>(&h2);
      }
      uint4* dst = reinterpret_cast<uint4*>(a.o + ((size_t)bh * a.N + row) * D + 32 * c);
#pragma unroll
      for (int i = 0; i < 4; ++i) dst[i] = make_uint4(out[4 * i], out[4 * i + 1], out[4 * i + 2], out[4 * i + 3]);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc<kTmemCols>(tmem);
}

// ---------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
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
bool make_map(CUtensorMap* m, const void* base, uint64_t dim0, uint64_t dim1, uint64_t dim2, uint32_t box0, uint32_t box1) {
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

template <int D>
cudaError_t run8(const Problem& pr, const QuantLayout& ql, const WorkLayout& wl, const uint8_t* quant,
                 void* o, uint8_t* work, cudaStream_t s) {
  alignas(64) CUtensorMap tq, tk, tv;
  if (!make_map(&tq, quant + ql.q_codes, D, pr.n_pad, pr.BH, D, 128) ||
      !make_map(&tk, quant + ql.k_codes, D, pr.n_pad, pr.BH, D, 128) ||
      !make_map(&tv, quant + ql.v_codes, pr.n_pad, D, pr.BH, 128, D))
    return cudaErrorUnknown;
  AttnArgs a{};
  a.q_scale = (const float*)(quant + ql.q_scale);
  a.k_scale = (const float*)(quant + ql.k_scale);
  a.v_scale = (const float*)(quant + ql.v_scale);
  a.v_means = (const __nv_bfloat16*)(quant + ql.v_means);
  a.o = (__nv_bfloat16*)o;
  a.status = (uint32_t*)(work + wl.status);
  a.N = pr.N; a.n_pad = pr.n_pad; a.nb = pr.nb; a.p_format = pr.p_format;
  a.sl = pr.softmax_scale * 1.4426950408889634f;
  a.code_off = 120.0f + pr.beta;
  const size_t smem = 1024 + 2 * 128 * D + D * 128 + D * 4 + 64;
  cudaError_t e = cudaFuncSetAttribute(attn_fwd_serial_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  attn_fwd_serial_kernel<D><<<dim3(pr.nb, pr.BH), 128, smem, s>>>(tq, tk, tv, a);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_attn_fwd(const Problem& pr, const QuantLayout& ql, const WorkLayout& wl,
                            const uint8_t* quant, void* o, uint8_t* work, cudaStream_t stream) {
  cudaError_t e = cudaMemsetAsync(work + wl.status, 0, 4, stream);
  if (e != cudaSuccess) return e;
  if (pr.bits != 8) return cudaErrorNotSupported;
  return pr.d == 128 ? run8<128>(pr, ql, wl, quant, o, work, stream) : run8<64>(pr, ql, wl, quant, o, work, stream);
}

}  // namespace vc
