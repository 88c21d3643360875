// Quantized attention forward of VC-Attention for sm_100a (Eq. 1, Eq. 6, Eq. 7).
//
// Two kernels share the arithmetic:
//   attn_fwd_2q_kernel      the default: warp-specialized, two 128-row query tiles per CTA,
//                           TMA ring for K^/R^ tiles, tcgen05 MMAs with accumulators in tensor
//                           memory, ExpCast-FP8 softmax warpgroups, correction warpgroups
//                           (described in front of the kernel)
//   attn_fwd_serial_kernel  one query tile per CTA, every step in program order behind
//                           __syncthreads; kept as an independent cross-check and for A/B timing
// Both read the bundle vc_prep writes: E4M3 codes of Q (query order), K (permuted order, row
// major) and the V residual (channel-major), per-block scales, per-channel value scale and the
// block means divided by it.  Epilogue: O = s_V * A / l, bf16, original query order.
#include <cuda_bf16.h>
#include <cuda_fp4.h>
#include <cuda_fp8.h>

#include "vc_internal.h"
#include "vc_sm100.cuh"
#include "vc_attn_shared.cuh"

namespace vc {
namespace {

using namespace sm100;
using namespace attn;


// Value of an ExpCast / E4M3 code in [0, 126] (non-negative): normals by placing the
// exponent and mantissa fields into an fp32 pattern, subnormals (codes 1..7) as m * 2^-9.
__device__ __forceinline__ float decode_pos_e4m3(uint32_t code) {
  return code >= 8u ? __uint_as_float((code + 960u) << 20) : (float)code * 0.001953125f;
}

// Serial kernel: TMA -> S = Q^ K^_j^T -> one thread per row (max, alpha, codes, row sum) ->
// P^ to tensor memory -> A = alpha A + r mu~_j on CUDA cores -> A += P^ R^_j, tile after tile.
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
// Two-query-tile kernel (default).  A CTA owns TWO 128-row query tiles of one (batch, head)
// and streams each K^_j / R^_j tile through both, so every key/value byte fetched from L2
// feeds 256 query rows.  Two decisions keep the softmax stage - the bottleneck on this GPU -
// as short as the method allows:
//   * The probability codes travel through SHARED memory, not through tensor memory, so a
//     score tile is free as soon as its 128 x 128 values are in registers; one score buffer
//     serves both query tiles in turn and S_t(j+1) is ready long before it is needed.
//   * The row sums of the decoded codes (Eq. 6: r_ij, and the normalizer l) come from the
//     tensor core: the value operand carries 16 extra rows of ones, so columns d..d+15 of the
//     accumulator hold l, rescaled by alpha together with the rest.  The softmax threads do
//     nothing but max, one fma.sat, one magic-number FMA and byte packing per score.
//
//   warp 0        TMA producer: Q0, Q1 once; then per key tile K^_j, R^_j and the tile's block
//                 mean (as a [d x 8] TF32 operand) through a 4-stage ring
//   warp 1        score issuer (one elected lane), per key tile j and query tile t:
//                   S    = Q^_t K^_j^T         4 x kind::f8f6f4, once the previous scores are read
//   warp 3        accumulator issuer, per key tile j and query tile t:
//                   A_t += P^_t(j) [R^_j | 1]  4 x kind::f8f6f4, N = d + 16, codes from shared memory
//                   A_t += rho_{j-1} mu~_{j-1} 1 x kind::tf32: the rank-one mean term of Eq. 6, one
//                                              tile late, because r_{j-1} is read back from A_t first
//   warps 4-7     softmax warpgroup of tile 0, one thread per query row (128 scores in
//   warps 8-11    registers); likewise tile 1: running max, alpha, ExpCast-FP8 codes (Eq. 7: no
//                 exponential, no conversion), code tile in the swizzled K-major layout
//   warps 12-15   correction warpgroup of tile 0 (16-19: tile 1), one thread per row: reads l
//                 back, r_{j-1} = l_{j-1} - alpha_{j-1} l_{j-2}, rescales A_t by alpha_j when a
//                 row maximum moved, hands (r_hi, r_lo) alpha_j to the mean MMA, writes the output
//
// Tensor memory: S (128 columns) | A_0 (d + 16) | A_1 (d + 16).
// P formats of the two-query-tile kernel
constexpr int kPfExpCast = 0, kPfExp = 1, kPfExpPoly = 2, kPfExpMix = 3;

// 2^x for x <= 8 without the special-function unit: x = n + f with n the nearest integer
// (1.5 * 2^23 trick) and |f| <= 1/2, 2^f by a degree-4 polynomial (relative error 3.7e-6, a
// 1/17000 of an E4M3 step), 2^n by an add into the exponent field.  Inputs below -24 give the
// value at -24, which rounds to code 0 like the exact result.
__device__ __forceinline__ float exp2_poly(float x) {
  x = fmaxf(x, -24.0f);
  const float t = x + 12582912.0f;
  const float f = x - (t - 12582912.0f);
  float p = fmaf(0.009676037356257439f, f, 0.05592203512787819f);
  p = fmaf(p, f, 0.2402210682630539f);
  p = fmaf(p, f, 0.6931210160255432f);
  p = fmaf(p, f, 1.0000001192092896f);
  return __uint_as_float(__float_as_uint(p) + (__float_as_uint(t) << 23));
}

template <int D, int PF, bool INT8>
__global__ void __launch_bounds__(640, 1)
attn_fwd_2q_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                   const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_mu,
                   const AttnArgs a) {
  constexpr int kTmemCols = 512;
  constexpr uint32_t O_COL = 128, O_STRIDE = 144, L_COL = D;   // A_t at O_COL + t * O_STRIDE; l in its column d
  // Register re-partition (setmaxnreg): the CTA owns 640 x 96 registers; a warpgroup that asks for
  // more than the others released would block forever, so the budget is checked at compile time.
  constexpr int kRegCtl = 48, kRegSoftmax = 160, kRegCorr = 56;
  static_assert(kRegCtl + 2 * kRegSoftmax + 2 * kRegCorr <= 5 * 96, "register budget exceeds the CTA's allocation");
  constexpr uint32_t kQBytes = 128 * D, kKBytes = 128 * D, kVBytes = D * 128, kOnesBytes = 16 * 128, kMuBytes = D * 32;
  constexpr uint32_t kStageBytes = kKBytes + kVBytes + kOnesBytes + ((kMuBytes + 1023) / 1024) * 1024;
  constexpr uint32_t kPBytes = 128 * 128, kAmBytes = 128 * 32;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char* sQ = smem;                                    // [2][128 x D]
  unsigned char* sP = smem + 2 * kQBytes;                      // [2][128 x 128] probability codes
  unsigned char* sAm = sP + 2 * kPBytes;                       // [2][128 x 8 fp32] row-sum pairs
  unsigned char* sStage = sAm + 2 * kAmBytes;                  // [kStages2]{K, V | ones, Mu}
  FaSmem* sh = reinterpret_cast<FaSmem*>(sStage + kStages2 * kStageBytes);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int qpair = blockIdx.x, bh = blockIdx.y;
  const int nb = a.nb;

  if (tid == 0) {
    mbar_init(&sh->q_full, 1);
    for (int i = 0; i < kStages2; ++i) { mbar_init(&sh->kv_full[i], 1); mbar_init(&sh->kv_empty[i], 2); }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&sh->s_full[i], 1); mbar_init(&sh->s_free[i], 128); mbar_init(&sh->o_done[i], 1);
      mbar_init(&sh->fin_full[i], 128); mbar_init(&sh->o_final[i], 1);
      for (int b = 0; b < 2; ++b) { mbar_init(&sh->a_full[i][b], 128); mbar_init(&sh->pc_full[i][b], 256); }
    }
    mbar_init(&sh->drain[0], 1); mbar_init(&sh->drain[1], 1);
    sh->abort = 0;
    sh->wait_limit = a.wait_limit;
    sh->wait_hint_ns = a.wait_hint_ns;
    mbar_fence_init();
    tma_prefetch_desc(&tm_q); tma_prefetch_desc(&tm_k); tma_prefetch_desc(&tm_v); tma_prefetch_desc(&tm_mu);
  }
  for (int i = tid; i < 2 * (int)kAmBytes / 16; i += 640) reinterpret_cast<uint4*>(sAm)[i] = make_uint4(0, 0, 0, 0);
  // 16 rows of E4M3 1.0 behind every value tile (the rows are uniform, so the swizzle is moot)
  for (int i = tid; i < kStages2 * (int)kOnesBytes / 4; i += 640)
    reinterpret_cast<uint32_t*>(sStage + (i / (kOnesBytes / 4)) * kStageBytes + kKBytes + kVBytes)[i % (kOnesBytes / 4)] = 0x38383838u;
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy stores -> tensor-core reads
  if (warp == 2) { tmem_alloc<kTmemCols>(&sh->tmem_base); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sh->tmem_base;
  const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);

  if (warp < 4) {
    reg_dec<kRegCtl>();
    if (warp == 0) {
      // ------------------------------------------------------------------ TMA producer
      // (the whole warp runs the loop; one elected lane issues the copies)
      if (elect_one()) {
        mbar_expect_tx(&sh->q_full, 2 * kQBytes);
        tma_load_3d(sQ, &tm_q, &sh->q_full, 0, (2 * qpair) * 128, bh);
        tma_load_3d(sQ + kQBytes, &tm_q, &sh->q_full, 0, (2 * qpair + 1) * 128, bh);   // past the end: zero fill
      }
      int j = 0;
      for (; j < nb; ++j) {
        const int st = j % kStages2, it = j / kStages2;
        unsigned char* base = sStage + st * kStageBytes;
        if (!warp_wait2(&sh->kv_empty[st], (it & 1) ^ 1, sh, a.status, 11)) break;
        if (elect_one()) {
          mbar_expect_tx(&sh->kv_full[st], kKBytes + kVBytes + kMuBytes);
          tma_load_3d(base, &tm_k, &sh->kv_full[st], 0, j * 128, bh);
          tma_load_3d(base + kKBytes, &tm_v, &sh->kv_full[st], j * 128, 0, bh);
          tma_load_3d(base + kKBytes + kVBytes + kOnesBytes, &tm_mu, &sh->kv_full[st], 0, 0, bh * nb + j);
        }
        __syncwarp();
      }
      drain_loads(sh, j);                                 // (returns at once on a normal run)
    } else if (warp == 1) {
      // ------------------------------------------------------------------ score issuer
      // Issues S_t = Q^_t K^_jT for both query tiles into the ONE score buffer, in the fixed order
      // S_0(0), S_1(0), S_0(1), S_1(1), ...: each may overwrite the buffer as soon as the previous
      // one has been read into registers.  (The whole warp runs the loop so that descriptors stay
      // in uniform registers; one elected lane issues.  A separate warp issues the A_t updates, so
      // that neither kind of MMA ever waits behind a barrier that only the other kind needs.)
      const uint32_t idesc_qk = INT8 ? idesc_s8(128, 128) : idesc_e4m3(128, 128);
      const uint64_t dq0 = smem_desc_kmajor(smem_u32(sQ), D), dq1 = smem_desc_kmajor(smem_u32(sQ + kQBytes), D);
      bool ok = warp_wait2(&sh->q_full, 0, sh, a.status, 20);
      for (int j = 0; ok && j < nb; ++j) {
        const int st = j % kStages2, it = j / kStages2;
        if (!(ok = warp_wait2(&sh->kv_full[st], it & 1, sh, a.status, 21))) break;
        const uint64_t dk = smem_desc_kmajor(smem_u32(sStage + st * kStageBytes), D);
#pragma unroll
        for (int t = 0; t < 2; ++t) {
          // S_0(j) waits for the read of S_1(j-1), S_1(j) for the read of S_0(j)
          if (t == 0 ? j > 0 : true) {
            if (!(ok = warp_wait2(&sh->s_free[1 - t], (t == 0 ? j - 1 : j) & 1, sh, a.status, 22))) break;
          }
          if (elect_one()) {
            tc_fence_after();
            const uint64_t dq = t == 0 ? dq0 : dq1;
#pragma unroll
            for (int k = 0; k < D / 32; ++k) {
              if constexpr (INT8) mma_s8_ss(tmem, dq + 2 * k, dk + 2 * k, idesc_qk, k > 0);
              else mma_f8_ss(tmem, dq + 2 * k, dk + 2 * k, idesc_qk, k > 0);
            }
            mma_commit(&sh->s_full[t]);
          }
          __syncwarp();
        }
      }
      drain_mmas(sh, 0);
    } else if (warp == 3) {
      // ------------------------------------------------------------------ accumulator issuer
      // A_t += P^_t(j) [R^_j | 1] once the codes are written, A_t is rescaled by alpha_j and the
      // row-sum pair of tile j-1 is in place; then the mean term of tile j-1.
      const uint32_t idesc_pv = idesc_e4m3(128, D + 16), idesc_mu = idesc_tf32(128, D);
      const uint64_t dp[2] = {smem_desc_kmajor(smem_u32(sP), 128), smem_desc_kmajor(smem_u32(sP + kPBytes), 128)};
      const uint64_t dam[2] = {smem_desc_kmajor(smem_u32(sAm), 32), smem_desc_kmajor(smem_u32(sAm + kAmBytes), 32)};
      bool ok = true;
      for (int j = 0; ok && j < nb; ++j) {
        const int st = j % kStages2, it = j / kStages2;
        const int stp = (j + kStages2 - 1) % kStages2;    // stage of tile j-1
        if (!(ok = warp_wait2(&sh->kv_full[st], it & 1, sh, a.status, 25))) break;
        const uint64_t dv = smem_desc_kmajor(smem_u32(sStage + st * kStageBytes + kKBytes), 128);
        const uint64_t dm = smem_desc_kmajor(smem_u32(sStage + stp * kStageBytes + kKBytes + kVBytes + kOnesBytes), 32);
#pragma unroll
        for (int t = 0; t < 2; ++t) {
          if (!(ok = warp_wait2(&sh->pc_full[t][j & 1], (j >> 1) & 1, sh, a.status, 23))) break;
          if (elect_one()) {
            tc_fence_after();
            const uint32_t o_col = tmem + O_COL + O_STRIDE * t;
#pragma unroll
            for (int k = 0; k < 4; ++k) mma_f8_ss(o_col, dp[t] + 2 * k, dv + 2 * k, idesc_pv, (j > 0) | (k > 0));
            if (j > 0) mma_tf32_ss(o_col, dam[t], dm, idesc_mu, 1);
            mma_commit(&sh->o_done[t]);
            if (j > 0) mma_commit(&sh->kv_empty[stp]);    // this tile is done with stage j-1
          }
          __syncwarp();
        }
      }
      const uint64_t dml = smem_desc_kmajor(smem_u32(sStage + ((nb - 1) % kStages2) * kStageBytes + kKBytes + kVBytes + kOnesBytes), 32);
#pragma unroll
      for (int t = 0; t < 2; ++t) {                       // mean term of the last tile
        if (!ok || !(ok = warp_wait2(&sh->fin_full[t], 0, sh, a.status, 27))) break;
        if (elect_one()) {
          tc_fence_after();
          mma_tf32_ss(tmem + O_COL + O_STRIDE * t, dam[t], dml, idesc_mu, 1);
          mma_commit(&sh->o_final[t]);
        }
        __syncwarp();
      }
      drain_mmas(sh, 1);
    }
  } else if (warp < 12) {
    // -------------------------------------------------------------------- softmax warpgroups
    reg_inc<kRegSoftmax>();
    const int t = (warp - 4) >> 2;                         // query tile of this warpgroup
    const int row = (warp & 3) * 32 + lane;
    const int qblk = 2 * qpair + t;
    // my row of the swizzled code tile: 16-byte chunk c sits at chunk position c ^ (row % 8)
    unsigned char* p_row = sP + t * kPBytes + (row >> 3) * 1024 + (row & 7) * 128;
    const float sq = qblk < nb ? a.q_scale[(size_t)bh * nb + qblk] : 1.0f;
    float m_run = -INFINITY;
    float sk_next = __ldg(&a.k_scale[(size_t)bh * nb]);   // fetched one tile ahead: an L2 round trip
    for (int j = 0; j < nb; ++j) {
      const int ph = j & 1;
      const float cs = (sq * sk_next) * a.sl;             // code units -> log2 domain
      if (j + 1 < nb) sk_next = __ldg(&a.k_scale[(size_t)bh * nb + j + 1]);
      if (!warp_wait2(&sh->s_full[t], ph, sh, a.status, 30)) break;
      tc_fence_after();
      uint32_t s0[32], s1[32], s2[32], s3[32];
      tmem_ld32(lane_base, s0); tmem_ld32(lane_base + 32, s1); tmem_ld32(lane_base + 64, s2); tmem_ld32(lane_base + 96, s3);
      tmem_wait_ld();
      tc_fence_before();
      mbar_arrive(&sh->s_free[t]);                        // the score buffer may be overwritten
      if constexpr (INT8) {
        // INT32 scores -> FP32, exactly: |s| <= 127 * 127 * 128 < 2^22, so the bits of 1.5 * 2^23 + s
        // are an integer add away, and subtracting the constant is exact.  (The two extra
        // instructions per score are what the E4M3 score product saves on this GPU.)
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          s0[i] = __float_as_uint(__uint_as_float(s0[i] + 0x4B400000u) - 12582912.0f);
          s1[i] = __float_as_uint(__uint_as_float(s1[i] + 0x4B400000u) - 12582912.0f);
          s2[i] = __float_as_uint(__uint_as_float(s2[i] + 0x4B400000u) - 12582912.0f);
          s3[i] = __float_as_uint(__uint_as_float(s3[i] + 0x4B400000u) - 12582912.0f);
        }
      }
      const int nv = a.N - j * 128;                       // >= 128 except on the ragged last tile
      if (nv < 128) {                                     // padded keys never win the maximum
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          if (i >= nv) s0[i] = 0xff800000u;
          if (32 + i >= nv) s1[i] = 0xff800000u;
          if (64 + i >= nv) s2[i] = 0xff800000u;
          if (96 + i >= nv) s3[i] = 0xff800000u;
        }
      }
      float mx[8];
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        mx[c] = max3(__uint_as_float(s0[16 * c]), __uint_as_float(s0[16 * c + 1]), __uint_as_float(s0[16 * c + 2]));
        mx[2 + c] = max3(__uint_as_float(s1[16 * c]), __uint_as_float(s1[16 * c + 1]), __uint_as_float(s1[16 * c + 2]));
        mx[4 + c] = max3(__uint_as_float(s2[16 * c]), __uint_as_float(s2[16 * c + 1]), __uint_as_float(s2[16 * c + 2]));
        mx[6 + c] = max3(__uint_as_float(s3[16 * c]), __uint_as_float(s3[16 * c + 1]), __uint_as_float(s3[16 * c + 2]));
#pragma unroll
        for (int i = 3; i < 15; i += 2) {
          mx[c] = max3(mx[c], __uint_as_float(s0[16 * c + i]), __uint_as_float(s0[16 * c + i + 1]));
          mx[2 + c] = max3(mx[2 + c], __uint_as_float(s1[16 * c + i]), __uint_as_float(s1[16 * c + i + 1]));
          mx[4 + c] = max3(mx[4 + c], __uint_as_float(s2[16 * c + i]), __uint_as_float(s2[16 * c + i + 1]));
          mx[6 + c] = max3(mx[6 + c], __uint_as_float(s3[16 * c + i]), __uint_as_float(s3[16 * c + i + 1]));
        }
        mx[c] = fmaxf(mx[c], __uint_as_float(s0[16 * c + 15]));
        mx[2 + c] = fmaxf(mx[2 + c], __uint_as_float(s1[16 * c + 15]));
        mx[4 + c] = fmaxf(mx[4 + c], __uint_as_float(s2[16 * c + 15]));
        mx[6 + c] = fmaxf(mx[6 + c], __uint_as_float(s3[16 * c + 15]));
      }
      const float mxa = max3(max3(mx[0], mx[1], mx[2]), max3(mx[3], mx[4], mx[5]), fmaxf(mx[6], mx[7]));
      const float m_new = fmaxf(m_run, mxa * cs);         // m' = max(m, rowmax S_ij)
      sh->alpha[t][row] = ex2_approx(m_run - m_new);      // alpha; 0 on the first tile
      mbar_arrive(&sh->a_full[t][j & 1]);
      m_run = m_new;
      // the previous code tile must have been consumed before it is overwritten
      if (j > 0 && !warp_wait2(&sh->o_done[t], (j - 1) & 1, sh, a.status, 31)) break;

      const float fa = cs * 0.0625f, fb = (a.code_off - 8.0f * m_new) * 0.0078125f, nm = 8.0f - m_new;
      const uint64_t fa2 = pack_f32x2(fa, fa), fb2 = pack_f32x2(fb, fb);
      auto code4 = [&](const uint32_t (&sv)[32], int w) -> uint32_t {
        if constexpr (PF == kPfExpCast) {
          // Eq. 7: t = (8 u + 120 + beta) / 128, code = round-to-nearest-even(128 t) clipped at 0
          // (two packed FP32 instructions and a saturating pack per two scores)
          return expcast_codes4(sv[4 * w], sv[4 * w + 1], sv[4 * w + 2], sv[4 * w + 3], fa2, fb2);
        } else {
          // exponentiate, then cast (Fig. 4a upper box): on the special-function unit, on the
          // FMA pipe by a polynomial, or three and one per word
          const float x0 = fmaf(__uint_as_float(sv[4 * w]), cs, nm), x1 = fmaf(__uint_as_float(sv[4 * w + 1]), cs, nm);
          const float x2 = fmaf(__uint_as_float(sv[4 * w + 2]), cs, nm), x3 = fmaf(__uint_as_float(sv[4 * w + 3]), cs, nm);
          float p0, p1, p2, p3;
          if constexpr (PF == kPfExp) {
            p0 = ex2_approx(x0); p1 = ex2_approx(x1); p2 = ex2_approx(x2); p3 = ex2_approx(x3);
          } else if constexpr (PF == kPfExpPoly) {
            p0 = exp2_poly(x0); p1 = exp2_poly(x1); p2 = exp2_poly(x2); p3 = exp2_poly(x3);
          } else {
            p0 = ex2_approx(x0); p1 = ex2_approx(x1); p2 = ex2_approx(x2); p3 = exp2_poly(x3);
          }
          const uint32_t lo = __nv_cvt_float2_to_fp8x2(make_float2(p0, p1), __NV_SATFINITE, __NV_E4M3);
          const uint32_t hi = __nv_cvt_float2_to_fp8x2(make_float2(p2, p3), __NV_SATFINITE, __NV_E4M3);
          return lo | (hi << 16);
        }
      };
      auto store16 = [&](const uint32_t (&sv)[32], int half, int chunk) {   // keys 16*chunk .. +15
        const uint4 v = make_uint4(code4(sv, 4 * half), code4(sv, 4 * half + 1), code4(sv, 4 * half + 2), code4(sv, 4 * half + 3));
        *reinterpret_cast<uint4*>(p_row + ((chunk ^ (row & 7)) << 4)) = v;
      };
      store16(s0, 0, 0); store16(s0, 1, 1); store16(s1, 0, 2); store16(s1, 1, 3);
      store16(s2, 0, 4); store16(s2, 1, 5); store16(s3, 0, 6); store16(s3, 1, 7);
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");          // my stores -> tensor-core reads
      mbar_arrive(&sh->pc_full[t][j & 1]);
    }
  } else {
    // -------------------------------------------------------------------- correction warpgroups
    reg_dec<kRegCorr>();
    const int t = (warp - 12) >> 2;
    const int row = (warp & 3) * 32 + lane;
    const int qblk = 2 * qpair + t;
    const uint32_t o_base = lane_base + O_COL + O_STRIDE * t;
    // my row of the row-sum operand: 32-byte rows, the two 16-byte chunks swap when (row / 4) is odd
    uint4* am_row = reinterpret_cast<uint4*>(sAm + t * kAmBytes + row * 32 + 16 * ((row >> 2) & 1));
    float l_resc = 0.f;       // l as it stands in column d after the latest rescale, before the tile's own sum
    float l_now = 0.f;
    bool ok = true;
    auto put_pair = [&](float rho) {                      // (rho_hi, rho_lo, 0, 0) for the mean MMA
      const uint32_t hi = (__float_as_uint(rho) + 0x1000u) & 0xffffe000u;   // nearest TF32
      *am_row = make_uint4(hi, __float_as_uint(rho - __uint_as_float(hi)), 0u, 0u);
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    };
    for (int j = 0; j < nb; ++j) {
      if (!(ok = warp_wait2(&sh->a_full[t][j & 1], (j >> 1) & 1, sh, a.status, 40))) break;
      const float alpha = sh->alpha[t][row];
      if (j > 0) {
        if (!(ok = warp_wait2(&sh->o_done[t], (j - 1) & 1, sh, a.status, 41))) break;
        tc_fence_after();
        l_now = __uint_as_float(tmem_ld1(o_base + L_COL));   // l after tile j-1
        tmem_wait_ld();
        const float r_prev = l_now - l_resc;                 // r_{j-1} = P~ 1 over the decoded codes
        if (__any_sync(0xffffffffu, alpha != 1.0f)) {        // a row maximum moved: A <- alpha A (l included)
          uint32_t r[16];
#pragma unroll 1
          for (int c = 0; c < D / 16; ++c) {
            tmem_ld16(o_base + 16 * c, r);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 16; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
            tmem_st16(o_base + 16 * c, r);
          }
          // of the 16 row-sum columns only column d is ever read, and its value is at hand
          tmem_st1(o_base + L_COL, __float_as_uint(l_now * alpha));
          tmem_wait_st();
          tc_fence_before();
        }
        l_resc = l_now * alpha;
        put_pair(r_prev * alpha);                            // added after the rescale, so referenced to m_j
      }
      mbar_arrive(&sh->pc_full[t][j & 1]);
    }
    // ---- last tile's mean term, then the epilogue: O = s_V * A / l
    if (ok && (ok = warp_wait2(&sh->o_done[t], (nb - 1) & 1, sh, a.status, 42))) {
      tc_fence_after();
      l_now = __uint_as_float(tmem_ld1(o_base + L_COL));
      tmem_wait_ld();
      put_pair(l_now - l_resc);
      mbar_arrive(&sh->fin_full[t]);
    }
    if (ok && warp_wait2(&sh->o_final[t], 0, sh, a.status, 43)) {
      tc_fence_after();
      const int grow = qblk * 128 + row;
      const float inv_l = 1.0f / l_now;
#pragma unroll 1
      for (int c = 0; c < D / 16; ++c) {
        uint32_t r[16];
        tmem_ld16(o_base + 16 * c, r);
        tmem_wait_ld();
        if (grow < a.N) {
          uint32_t out[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float x0 = __uint_as_float(r[2 * i]) * inv_l * __ldg(&a.v_scale[(size_t)bh * D + 16 * c + 2 * i]);
            const float x1 = __uint_as_float(r[2 * i + 1]) * inv_l * __ldg(&a.v_scale[(size_t)bh * D + 16 * c + 2 * i + 1]);
            __nv_bfloat162 h2 = __floats2bfloat162_rn(x0, x1);
            out[i] = *reinterpret_cast<uint32_t*>(&h2);
          }
          uint4* dst = reinterpret_cast<uint4*>(a.o + ((size_t)bh * a.N + grow) * D + 16 * c);
          dst[0] = make_uint4(out[0], out[1], out[2], out[3]);
          dst[1] = make_uint4(out[4], out[5], out[6], out[7]);
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 2) tmem_dealloc<kTmemCols>(tmem);
}

// ---------------------------------------------------------------------------------------
// 4-bit path (NVFP4 Q, K, R and P; App. A "Scope of ExpCast-FP8", App. B).
//
// An E2M1 element times its E4M3 microscale has at most six significant bits, so it is exact
// in bf16: the operands are expanded once per call into bf16 tiles and the two products run as
// kind::f16 MMAs with FP32 accumulation - bit-for-bit the arithmetic of a block-scaled FP4 MMA.
// The probability tile is quantized to NVFP4 in the softmax stage (per row and 16 keys: E4M3
// microscale of max p / 6, E2M1 elements) and handed to the tensor core as the exact bf16
// values of those codes.  This kernel is the simple serial form (one query tile per CTA, every
// step behind __syncthreads); the paper itself declines a 4-bit datacenter configuration
// because the per-16 scale computation sits on the softmax critical path.
__global__ void nvfp4_expand_kernel(const uint8_t* __restrict__ codes, const uint8_t* __restrict__ micro,
                                    __nv_bfloat16* __restrict__ out, size_t n_groups) {
  const size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x;   // one group of 16 elements
  if (g >= n_groups) return;
  const uint2 c = *reinterpret_cast<const uint2*>(codes + g * 8);
  const __half_raw hs = __nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)micro[g], __NV_E4M3);
  const float sdec = __half2float(__half(hs));
  const uint32_t w[2] = {c.x, c.y};
  uint32_t o[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const __half2_raw h2 = __nv_cvt_fp4x2_to_halfraw2((__nv_fp4x2_storage_t)((w[i >> 2] >> (8 * (i & 3))) & 0xffu), __NV_E2M1);
    const float2 f = __half22float2(__half2(h2));
    __nv_bfloat162 b = __floats2bfloat162_rn(f.x * sdec, f.y * sdec);
    o[i] = *reinterpret_cast<uint32_t*>(&b);
  }
  uint4* dst = reinterpret_cast<uint4*>(out + g * 16);
  dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
  dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
}

struct Attn4Args {
  const float *q_g, *k_g;          // NVFP4 outer scales per (b, h)
  const __nv_bfloat16* v_means;    // unscaled block means
  __nv_bfloat16* o;
  uint32_t* status;
  int N, n_pad, nb;
  float sl;
};

template <int D>
__global__ void __launch_bounds__(128)
attn_fwd_serial4_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                        const __grid_constant__ CUtensorMap tm_v, const Attn4Args a) {
  constexpr int kTmemCols = 512;
  constexpr uint32_t S_COL = 0, P_COL = 128, O_COL = 256;
  constexpr int kQH = D / 64;                        // 128-byte column halves of a Q/K tile
  constexpr uint32_t kHalfQ = 128 * 128, kHalfV = D * 128;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char* sQ = smem;                          // [kQH][128 rows x 128 B]
  unsigned char* sK = sQ + kQH * kHalfQ;             // [kQH][128 rows x 128 B]
  unsigned char* sV = sK + kQH * kHalfQ;             // [2][D rows x 128 B]: tokens 0..63, 64..127
  float* sMu = reinterpret_cast<float*>(sV + 2 * kHalfV);
  uint64_t* bars = reinterpret_cast<uint64_t*>(sMu + D);
  uint64_t *bar_q = bars, *bar_kv = bars + 1, *bar_s = bars + 2, *bar_o = bars + 3;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 4);

  const int tid = threadIdx.x, warp = tid >> 5;
  const int qblk = blockIdx.x, bh = blockIdx.y;
  bool alive = true;

  if (tid == 0) {
    mbar_init(bar_q, 1); mbar_init(bar_kv, 1); mbar_init(bar_s, 1); mbar_init(bar_o, 1);
    mbar_fence_init();
  }
  if (warp == 0) { tmem_alloc<kTmemCols>(tmem_slot); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);

  if (tid == 0) {
    mbar_expect_tx(bar_q, kQH * kHalfQ);
    for (int h = 0; h < kQH; ++h) tma_load_3d(sQ + h * kHalfQ, &tm_q, bar_q, 128 * h, qblk * 128, bh);
  }
  if (!mbar_wait(bar_q, 0)) { alive = false; atomicExch(a.status, kErrTimeout | 1); }

  const float cs = (a.q_g[bh] * a.k_g[bh]) * a.sl;   // code units -> log2 domain
  const uint32_t idesc_qk = idesc_bf16(128, 128), idesc_pv = idesc_bf16(128, D);
  float m_run = -INFINITY, l_run = 0.f;
  for (int j = 0; j < a.nb; ++j) {
    const uint32_t ph = j & 1;
    if (tid == 0) {
      mbar_expect_tx(bar_kv, kQH * kHalfQ + 2 * kHalfV);
      for (int h = 0; h < kQH; ++h) tma_load_3d(sK + h * kHalfQ, &tm_k, bar_kv, 128 * h, j * 128, bh);
      for (int h = 0; h < 2; ++h) tma_load_3d(sV + h * kHalfV, &tm_v, bar_kv, 2 * (j * 128 + 64 * h), 0, bh);
    }
    if (tid < D / 2) {
      const __nv_bfloat162 m2 = *reinterpret_cast<const __nv_bfloat162*>(a.v_means + ((size_t)bh * a.nb + j) * D + 2 * tid);
      sMu[2 * tid] = __low2float(m2);
      sMu[2 * tid + 1] = __high2float(m2);
    }
    if (alive && !mbar_wait(bar_kv, ph)) { alive = false; atomicExch(a.status, kErrTimeout | 2); }
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
      for (int h = 0; h < kQH; ++h) {
        const uint64_t dq = smem_desc_kmajor(smem_u32(sQ + h * kHalfQ), 128), dk = smem_desc_kmajor(smem_u32(sK + h * kHalfQ), 128);
#pragma unroll
        for (int k = 0; k < 4; ++k) mma_f16_ss(tmem + S_COL, dq + 2 * k, dk + 2 * k, idesc_qk, (h > 0) | (k > 0));
      }
      mma_commit(bar_s);
    }
    if (alive && !mbar_wait(bar_s, ph)) { alive = false; atomicExch(a.status, kErrTimeout | 3); }
    tc_fence_after();

    // ---- softmax stage: this thread owns query row 32*warp + lane
    const int nv = min(128, a.N - j * 128);
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
    const float m_new = fmaxf(m_run, mx * cs);
    const float alpha = exp2f(m_run - m_new);
    float rsum = 0.f;
#pragma unroll 1
    for (int c = 0; c < 4; ++c) {
      tmem_ld32(lane_base + S_COL + 32 * c, r);
      tmem_wait_ld();
      uint32_t pk[16];
#pragma unroll
      for (int g = 0; g < 2; ++g) {                   // NVFP4 group of 16 keys
        float p[16], gmax = 0.f;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const int key = 32 * c + 16 * g + i;
          const float u = fmaf(__uint_as_float(r[16 * g + i]), cs, -m_new);
          p[i] = key < nv ? exp2f(u) * 2688.0f : 0.f;   // the row maximum maps to 6 * 448
          gmax = fmaxf(gmax, p[i]);
        }
        const uint32_t sb = __nv_cvt_float_to_fp8(gmax * (1.0f / 6.0f), __NV_SATFINITE, __NV_E4M3);
        const __half_raw hs = __nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)sb, __NV_E4M3);
        const float sdec = __half2float(__half(hs));
        const float rcp = sdec > 0.f ? 1.0f / sdec : 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const __nv_fp4x2_storage_t two = __nv_cvt_float2_to_fp4x2(make_float2(p[2 * i] * rcp, p[2 * i + 1] * rcp), __NV_E2M1, cudaRoundNearest);
          const __half2_raw h2 = __nv_cvt_fp4x2_to_halfraw2(two, __NV_E2M1);
          const float2 f = __half22float2(__half2(h2));
          const float p0 = f.x * sdec, p1 = f.y * sdec;     // decoded probabilities, exact in bf16
          rsum += p0 + p1;
          __nv_bfloat162 b = __floats2bfloat162_rn(p0, p1);
          pk[8 * g + i] = *reinterpret_cast<uint32_t*>(&b);
        }
      }
      uint32_t lo[8], hi[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) { lo[i] = pk[i]; hi[i] = pk[8 + i]; }
      tmem_st8(lane_base + P_COL + 16 * c, lo);
      tmem_st8(lane_base + P_COL + 16 * c + 8, hi);
    }
    l_run = alpha * l_run + rsum;
    m_run = m_new;

    // ---- A <- alpha A + r mu_j (means unscaled at 4 bits, App. B); the product follows
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
      for (int h = 0; h < 2; ++h) {
        const uint64_t dv = smem_desc_kmajor(smem_u32(sV + h * kHalfV), 128);
#pragma unroll
        for (int k = 0; k < 4; ++k) mma_f16_ts(tmem + O_COL, tmem + P_COL + 32 * h + 8 * k, dv + 2 * k, idesc_pv, 1);
      }
      mma_commit(bar_o);
    }
    if (alive && !mbar_wait(bar_o, ph)) { alive = false; atomicExch(a.status, kErrTimeout | 4); }
    tc_fence_after();
  }

  // ---- epilogue: O = A / l
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
        __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(r[2 * i]) * inv_l, __uint_as_float(r[2 * i + 1]) * inv_l);
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
  a.wait_limit = attn_wait_limit();
  a.wait_hint_ns = attn_wait_hint_ns();
  cudaError_t e;
  if (pr.kernel_variant == 1) {     // serial reference kernel
    const size_t smem = 1024 + 2 * 128 * D + D * 128 + D * 4 + 64;
    if ((e = cudaFuncSetAttribute(attn_fwd_serial_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
    attn_fwd_serial_kernel<D><<<dim3(pr.nb, pr.BH), 128, smem, s>>>(tq, tk, tv, a);
    count_launches(1);
    return cudaGetLastError();
  }
  if (pr.kernel_variant == 0) {     // two query tiles per CTA (default)
    alignas(64) CUtensorMap tmt;
    if (!make_map(&tmt, work + wl.mu_mma, 32, D, (uint64_t)pr.BH * pr.nb, 32, D)) return cudaErrorUnknown;
    const size_t n = (size_t)pr.BH * pr.nb * D;
    means_tile_layout_kernel<D><<<(unsigned)((n + 255) / 256), 256, 0, s>>>(a.v_means, (float*)(work + wl.mu_mma), n);
    const size_t stage = 2 * 128 * D + 2048 + ((D * 32 + 1023) / 1024) * 1024;
    const size_t smem2 = 1024 + 2 * 128 * D + 2 * 128 * 128 + 2 * 128 * 32 + kStages2 * stage + sizeof(FaSmem);
    const dim3 grid((pr.nb + 1) / 2, pr.BH);
    const bool int8 = pr.flags & VC_FLAG_INT8_QK;
#define VC_LAUNCH_2Q(EC, I8)                                                                                             \
  {                                                                                                                      \
    if ((e = cudaFuncSetAttribute(attn_fwd_2q_kernel<D, EC, I8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem2)) != cudaSuccess) return e; \
    attn_fwd_2q_kernel<D, EC, I8><<<grid, 640, smem2, s>>>(tq, tk, tv, tmt, a);                                           \
  }
    const int pf = pr.p_format == VC_P_EXPCAST_E4M3 ? kPfExpCast
                   : pr.p_format == VC_P_EXP_E4M3   ? kPfExp
                   : pr.p_format == VC_P_EXP_POLY_E4M3 ? kPfExpPoly : kPfExpMix;
    if (int8) {
      if (pf == kPfExpCast) VC_LAUNCH_2Q(kPfExpCast, true)
      else if (pf == kPfExp) VC_LAUNCH_2Q(kPfExp, true)
      else return cudaErrorNotSupported;
    } else {
      if (pf == kPfExpCast) VC_LAUNCH_2Q(kPfExpCast, false)
      else if (pf == kPfExp) VC_LAUNCH_2Q(kPfExp, false)
      else if (pf == kPfExpPoly) VC_LAUNCH_2Q(kPfExpPoly, false)
      else VC_LAUNCH_2Q(kPfExpMix, false)
    }
#undef VC_LAUNCH_2Q
    count_launches(2);
    return cudaGetLastError();
  }
  return cudaErrorNotSupported;
}

template <int D>
cudaError_t run4(const Problem& pr, const QuantLayout& ql, const WorkLayout& wl, const uint8_t* quant,
                 void* o, uint8_t* work, cudaStream_t s) {
  // expand NVFP4 codes x microscales to bf16 tiles in the workspace
  const size_t elems = (size_t)pr.BH * pr.n_pad * D, groups = elems / 16;
  __nv_bfloat16* qb = reinterpret_cast<__nv_bfloat16*>(work + wl.expand);
  __nv_bfloat16 *kb = qb + elems, *vb = kb + elems;
  const unsigned blocks = (unsigned)((groups + 255) / 256);
  nvfp4_expand_kernel<<<blocks, 256, 0, s>>>(quant + ql.q_codes, quant + ql.q_micro, qb, groups);
  nvfp4_expand_kernel<<<blocks, 256, 0, s>>>(quant + ql.k_codes, quant + ql.k_micro, kb, groups);
  nvfp4_expand_kernel<<<blocks, 256, 0, s>>>(quant + ql.v_codes, quant + ql.v_micro, vb, groups);
  alignas(64) CUtensorMap tq, tk, tv;
  if (!make_map(&tq, qb, (uint64_t)D * 2, pr.n_pad, pr.BH, 128, 128) ||
      !make_map(&tk, kb, (uint64_t)D * 2, pr.n_pad, pr.BH, 128, 128) ||
      !make_map(&tv, vb, (uint64_t)pr.n_pad * 2, D, pr.BH, 128, D))
    return cudaErrorUnknown;
  Attn4Args a{};
  a.q_g = (const float*)(quant + ql.q_scale);
  a.k_g = (const float*)(quant + ql.k_scale);
  a.v_means = (const __nv_bfloat16*)(quant + ql.v_means);
  a.o = (__nv_bfloat16*)o;
  a.status = (uint32_t*)(work + wl.status);
  a.N = pr.N; a.n_pad = pr.n_pad; a.nb = pr.nb;
  a.sl = pr.softmax_scale * 1.4426950408889634f;
  const size_t smem = 1024 + 2 * (D / 64) * 128 * 128 + 2 * D * 128 + D * 4 + 64;
  cudaError_t e = cudaFuncSetAttribute(attn_fwd_serial4_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  attn_fwd_serial4_kernel<D><<<dim3(pr.nb, pr.BH), 128, smem, s>>>(tq, tk, tv, a);
  count_launches(4);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_attn_fwd(const Problem& pr, const QuantLayout& ql, const WorkLayout& wl,
                            const uint8_t* quant, void* o, uint8_t* work, cudaStream_t stream, bool clear_status) {
  if (clear_status) {
    cudaError_t e = cudaMemsetAsync(work + wl.status, 0, 4, stream);
    if (e != cudaSuccess) return e;
  }
  if (pr.bits == 4 && pr.kernel_variant == 0) return launch_attn_fwd4(pr, ql, wl, quant, o, work, stream);
  if (pr.bits == 4) return pr.d == 128 ? run4<128>(pr, ql, wl, quant, o, work, stream) : run4<64>(pr, ql, wl, quant, o, work, stream);
  return pr.d == 128 ? run8<128>(pr, ql, wl, quant, o, work, stream) : run8<64>(pr, ql, wl, quant, o, work, stream);
}

}  // namespace vc
