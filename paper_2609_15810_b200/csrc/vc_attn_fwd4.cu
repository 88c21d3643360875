// 4-bit attention forward of VC-Attention on block-scaled FP4 tensor-core instructions
// (App. A "Scope of ExpCast-FP8", App. B: NVFP4 Q, K, R and P).
//
// Every operand of both products is NVFP4 as vc_prep wrote it - E2M1 elements, two per byte,
// under an unsigned E4M3 factor per 16 elements along the contraction axis - and both products
// run as tcgen05.mma kind::mxf4nvf4 (K = 64 per instruction), which multiplies each 16-element
// partial sum by the two factors.  The factors live in tensor memory; tcgen05.cp brings them
// there from shared memory in 512-byte chunks (128 operand rows x 4 groups).  A small pre-pass
// rewrites the bundle's row-major factor arrays into that chunk order, per 128-row tile.
//
// The pipeline is the one of the 8-bit kernel (two query tiles per CTA, one shared score
// buffer, probability codes through shared memory, the row sums l from 16 rows of ones behind
// the value tile, the block-mean term as a TF32 MMA one tile late).  What differs is the
// softmax stage: P is quantized to NVFP4 per row and 16 keys.  The group maxima are a
// by-product of the running-max pass; per group the E4M3 factor of max p / 6 is formed once,
// its log2 is folded into the exponent offset, and every element costs one FMA, one ex2 and
// half a conversion:  code = E2M1(2^(s cs + log2 2688 - m' - log2 f_g)).  (Moving part of the
// exponentials to a polynomial on the FMA pipe was measured and is slower: the stage is bound by
// issue slots and hand-off latency before the special-function unit, which runs at 64 %.)
//
// HYB = true is the hybrid 4-bit arrangement: the score product stays NVFP4, but P is the
// ExpCast-FP8 code of Eq. 7 (two FMAs per score, as in the 8-bit kernel) and the value product
// runs as kind::mxf8f6f4: E4M3 P^ times E2M1 R^ under power-of-two factors per 32 tokens.  The
// value tile arrives through a 4-bit tensor map that spreads it into the 16-byte containers
// that instruction kind reads; P^ carries the constant factor 1.
#include <cuda_bf16.h>
#include <cuda_fp8.h>

#include "vc_attn_shared.cuh"
#include "vc_internal.h"
#include "vc_sm100.cuh"

namespace vc {
namespace {

using namespace sm100;
using namespace attn;

// Factor arrays -> MMA chunk order.  One CTA per (b, h, 128-row tile), thread r = operand row.
//   sf_q  [BH*nb][D/64][512]          Q^ factors of query tile
//   sf_kv [BH*nb][D/64 + 2][512]      K^ factors of key tile, then the R^ factors of the same
//                                     tile (operand rows = channels, groups = 16 tokens);
//                                     HYB: [D/64 + 1] chunks, the last one holding the four
//                                     power-of-two factors (32 tokens each) of every channel
// Chunk byte 16 (r % 32) + 4 (r / 32) + k  <-  factor of row r, group 4 kb + k.
template <int D, bool HYB>
__global__ void __launch_bounds__(128)
nvfp4_sf_tiles_kernel(const uint8_t* __restrict__ q_micro, const uint8_t* __restrict__ k_micro,
                      const uint8_t* __restrict__ v_micro, uint8_t* __restrict__ sf_q, uint8_t* __restrict__ sf_kv,
                      int nb, int n_pad) {
  constexpr int KB = D / 64, NVC = HYB ? 1 : 2;
  const int tile = blockIdx.x, bh = blockIdx.y, r = threadIdx.x;
  const size_t t_idx = (size_t)bh * nb + tile;
  const uint32_t pos = (r & 31) * 16 + (r >> 5) * 4;
  const size_t row = (size_t)bh * n_pad + (size_t)tile * 128 + r;
  const uint32_t* qm = reinterpret_cast<const uint32_t*>(q_micro + row * (D / 16));
  const uint32_t* km = reinterpret_cast<const uint32_t*>(k_micro + row * (D / 16));
#pragma unroll
  for (int kb = 0; kb < KB; ++kb) {
    *reinterpret_cast<uint32_t*>(sf_q + t_idx * (KB * 512) + kb * 512 + pos) = qm[kb];
    *reinterpret_cast<uint32_t*>(sf_kv + t_idx * ((KB + NVC) * 512) + kb * 512 + pos) = km[kb];
  }
  if constexpr (HYB) {
    uint32_t w = 0;
    if (r < D) w = *reinterpret_cast<const uint32_t*>(v_micro + ((size_t)bh * D + r) * (n_pad / 32) + (size_t)tile * 4);
    else if (r < D + 16) w = 0x7f7f7f7fu;   // the rows of ones: factor 2^0
    *reinterpret_cast<uint32_t*>(sf_kv + t_idx * ((KB + NVC) * 512) + KB * 512 + pos) = w;
    return;
  }
  uint32_t w0 = 0, w1 = 0;
  if (r < D) {
    const uint2 vm = *reinterpret_cast<const uint2*>(v_micro + ((size_t)bh * D + r) * (n_pad / 16) + (size_t)tile * 8);
    w0 = vm.x; w1 = vm.y;
  } else if (r < D + 16) {
    w0 = w1 = 0x38383838u;   // the rows of ones behind the value tile carry the factor 1.0
  }
  uint8_t* dst = sf_kv + t_idx * ((KB + 2) * 512) + KB * 512 + pos;
  *reinterpret_cast<uint32_t*>(dst) = w0;
  *reinterpret_cast<uint32_t*>(dst + 512) = w1;
}

struct Attn4Args {
  const float *q_g, *k_g;          // NVFP4 outer scales per (b, h)
  const uint8_t *sf_q, *sf_kv;     // factor chunks (see nvfp4_sf_tiles_kernel)
  __nv_bfloat16* o;
  uint32_t* status;
  int N, n_pad, nb;
  float sl;                        // softmax_scale * log2(e)
  float code_off;                  // 120 + beta  (Eq. 7; hybrid arrangement only)
  uint32_t wait_limit;             // polls after which a wait gives up
  uint32_t wait_hint_ns;
};

// Value of a non-negative E4M3 byte.
__device__ __forceinline__ float decode_ue4m3(uint32_t code) {
  return code >= 8u ? __uint_as_float((code + 960u) << 20) : (float)code * 0.001953125f;
}

//   warp 0        TMA producer: Q^ tiles and their factors once; per key tile K^_j, R^_j, the
//                 tile's factor chunks and block mean through a 4-stage ring
//   warp 1        score issuer:        S = Q^_t K^_j^T            D/64 x kind::mxf4nvf4
//   warp 3        accumulator issuer:  A_t += P^_t(j) [R^_j | 1]  2 x kind::mxf4nvf4, N = d + 16
//                                      A_t += rho_{j-1} mu_{j-1}  1 x kind::tf32
//   warps 4-11    softmax warpgroups (tile 0, tile 1), one thread per query row
//   warps 12-19   correction warpgroups, one thread per query row
// Tensor memory: S (128 columns) | A_0 (d + 16) | A_1 (d + 16) | scale factors (56 columns).
template <int D, bool HYB>
__global__ void __launch_bounds__(640, 1)
attn4_fwd_2q_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_mu,
                    const Attn4Args a) {
  constexpr int kTmemCols = 512;
  constexpr int KB = D / 64;                        // K = 64 steps of the score product
  constexpr int kRowB = D / 2;                      // bytes per Q^/K^ row
  constexpr uint32_t O_COL = 128, O_STRIDE = 144, L_COL = D;
  constexpr uint32_t SF_COL = 416;
  constexpr uint32_t SFQ_COL = SF_COL, SFK_COL = SF_COL + 16, SFP_COL = SF_COL + 24, SFV_COL = SF_COL + 40;
  constexpr int kRegCtl = 48, kRegSoftmax = 160, kRegCorr = 56;
  static_assert(kRegCtl + 2 * kRegSoftmax + 2 * kRegCorr <= 5 * 96, "register budget exceeds the CTA's allocation");
  constexpr int NVC = HYB ? 1 : 2;                  // value factor chunks per key tile
  constexpr uint32_t kVRow = HYB ? 128 : 64;        // bytes of a value row in shared memory
  constexpr uint32_t kQBytes = 128 * kRowB, kKBytes = 128 * kRowB, kVBytes = D * kVRow, kOnesBytes = 16 * kVRow;
  constexpr uint32_t kVTx = D * 64;                 // bytes the value copy reports (the packed ones)
  constexpr uint32_t kMuBytes = D * 32, kMuPad = ((kMuBytes + 1023) / 1024) * 1024;
  constexpr uint32_t kSfqBytes = KB * 512, kSfBytes = (KB + NVC) * 512, kSfPad = ((kSfBytes + 1023) / 1024) * 1024;
  constexpr uint32_t kStageBytes = kKBytes + kVBytes + kOnesBytes + kMuPad + kSfPad;
  constexpr uint32_t kPBytes = 128 * kVRow, kSfpBytes = 1024, kAmBytes = 128 * 32;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char* sQ = smem;                                    // [2][128 x D/2]
  unsigned char* sP = sQ + 2 * kQBytes;                        // [2][128 x 64] probability codes (HYB: 128 x 128)
  unsigned char* sAm = sP + 2 * kPBytes;                       // [2][128 x 8 fp32] row-sum pairs
  unsigned char* sSfq = sAm + 2 * kAmBytes;                    // [2][KB][512] Q^ factors
  unsigned char* sSfp = sSfq + 2 * 1024;                       // [2][2][512]  P^ factors (HYB: one chunk of ones)
  unsigned char* sSfOnes = sSfp + 2 * kSfpBytes;               // [512] factors of value rows 128..143
  unsigned char* sStage = sSfOnes + 1024;                      // [kStages2]{K, V | ones, Mu, factors}
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
  // 16 rows of E2M1 1.0 (two per byte) behind every value tile; their factor chunk: 1.0 for
  // rows 0..15 of the second 128-row half, group bytes 0..3
  // (HYB: the same bytes, of which the product reads the low 8 of every 16; factor code 127 = 2^0,
  // and a chunk of that code for every row of P^)
  for (int i = tid; i < kStages2 * (int)kOnesBytes / 4; i += 640)
    reinterpret_cast<uint32_t*>(sStage + (i / (kOnesBytes / 4)) * kStageBytes + kKBytes + kVBytes)[i % (kOnesBytes / 4)] = 0x22222222u;
  for (int i = tid; i < 128; i += 640)
    reinterpret_cast<uint32_t*>(sSfOnes)[i] = ((i & 3) == 0 && i < 64) ? (HYB ? 0x7f7f7f7fu : 0x38383838u) : 0u;
  if constexpr (HYB)
    for (int i = tid; i < 128; i += 640) reinterpret_cast<uint32_t*>(sSfp)[i] = 0x7f7f7f7fu;
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
      if (elect_one()) {
        mbar_expect_tx(&sh->q_full, 2 * kQBytes + 2 * kSfqBytes);
        for (int t = 0; t < 2; ++t) {
          const int qb = 2 * qpair + t;                    // past the end: zero codes, any factors
          tma_load_3d(sQ + t * kQBytes, &tm_q, &sh->q_full, 0, qb * 128, bh);
          bulk_load(sSfq + t * 1024, a.sf_q + ((size_t)bh * nb + min(qb, nb - 1)) * kSfqBytes, kSfqBytes, &sh->q_full);
        }
      }
      int j = 0;
      for (; j < nb; ++j) {
        const int st = j % kStages2, it = j / kStages2;
        unsigned char* base = sStage + st * kStageBytes;
        if (!warp_wait2(&sh->kv_empty[st], (it & 1) ^ 1, sh, a.status, 11)) break;
        if (elect_one()) {
          mbar_expect_tx(&sh->kv_full[st], kKBytes + kVTx + kMuBytes + kSfBytes);
          tma_load_3d(base, &tm_k, &sh->kv_full[st], 0, j * 128, bh);
          tma_load_3d(base + kKBytes, &tm_v, &sh->kv_full[st], HYB ? j * 128 : j * 64, 0, bh);   // elements resp. bytes
          tma_load_3d(base + kKBytes + kVBytes + kOnesBytes, &tm_mu, &sh->kv_full[st], 0, 0, bh * nb + j);
          bulk_load(base + kKBytes + kVBytes + kOnesBytes + kMuPad, a.sf_kv + ((size_t)bh * nb + j) * kSfBytes, kSfBytes,
                    &sh->kv_full[st]);
        }
        __syncwarp();
      }
      drain_loads(sh, j);                                 // (returns at once on a normal run)
    } else if (warp == 1) {
      // ------------------------------------------------------------------ score issuer
      const uint32_t idesc_qk = idesc_nvfp4(128, 128);
      const uint64_t dq0 = smem_desc_kmajor(smem_u32(sQ), kRowB), dq1 = smem_desc_kmajor(smem_u32(sQ + kQBytes), kRowB);
      bool ok = warp_wait2(&sh->q_full, 0, sh, a.status, 20);
      if (ok && elect_one()) {
        for (int t = 0; t < 2; ++t)
          for (int kb = 0; kb < KB; ++kb)
            tmem_cp_sf(tmem + SFQ_COL + (t * KB + kb) * 4, smem_desc_sf_chunk(smem_u32(sSfq + t * 1024 + kb * 512)));
      }
      __syncwarp();
      for (int j = 0; ok && j < nb; ++j) {
        const int st = j % kStages2, it = j / kStages2;
        if (!(ok = warp_wait2(&sh->kv_full[st], it & 1, sh, a.status, 21))) break;
        const unsigned char* base = sStage + st * kStageBytes;
        const uint64_t dk = smem_desc_kmajor(smem_u32(base), kRowB);
        const uint32_t sf_smem = smem_u32(base + kKBytes + kVBytes + kOnesBytes + kMuPad);
#pragma unroll
        for (int t = 0; t < 2; ++t) {
          if (t == 0 ? j > 0 : true) {
            if (!(ok = warp_wait2(&sh->s_free[1 - t], (t == 0 ? j - 1 : j) & 1, sh, a.status, 22))) break;
          }
          if (elect_one()) {
            tc_fence_after();
            if (t == 0) {
#pragma unroll
              for (int kb = 0; kb < KB; ++kb) tmem_cp_sf(tmem + SFK_COL + kb * 4, smem_desc_sf_chunk(sf_smem + kb * 512));
            }
            const uint64_t dq = t == 0 ? dq0 : dq1;
#pragma unroll
            for (int kb = 0; kb < KB; ++kb)
              mma_nvfp4_ss(tmem, dq + 2 * kb, dk + 2 * kb, idesc_qk, kb > 0, tmem + SFQ_COL + (t * KB + kb) * 4,
                           tmem + SFK_COL + kb * 4);
            mma_commit(&sh->s_full[t]);
          }
          __syncwarp();
        }
      }
      drain_mmas(sh, 0);
    } else if (warp == 3) {
      // ------------------------------------------------------------------ accumulator issuer
      const uint32_t idesc_pv = idesc_nvfp4(128, D + 16), idesc_mu = idesc_tf32(128, D);
      const uint64_t dp[2] = {smem_desc_kmajor(smem_u32(sP), kVRow), smem_desc_kmajor(smem_u32(sP + kPBytes), kVRow)};
      const uint64_t dam[2] = {smem_desc_kmajor(smem_u32(sAm), 32), smem_desc_kmajor(smem_u32(sAm + kAmBytes), 32)};
      if (elect_one()) {
        if (D == 128) {                                    // factors of the rows of ones (value rows 128..143)
          tmem_cp_sf(tmem + SFV_COL + 4, smem_desc_sf_chunk(smem_u32(sSfOnes)));
          if (!HYB) tmem_cp_sf(tmem + SFV_COL + 12, smem_desc_sf_chunk(smem_u32(sSfOnes)));
        }
        if (HYB) tmem_cp_sf(tmem + SFP_COL, smem_desc_sf_chunk(smem_u32(sSfp)));   // P^: factor 1 everywhere
      }
      __syncwarp();
      bool ok = true;
      for (int j = 0; ok && j < nb; ++j) {
        const int st = j % kStages2, it = j / kStages2;
        const int stp = (j + kStages2 - 1) % kStages2;    // stage of tile j-1
        if (!(ok = warp_wait2(&sh->kv_full[st], it & 1, sh, a.status, 25))) break;
        const unsigned char* base = sStage + st * kStageBytes;
        const uint64_t dv = smem_desc_kmajor(smem_u32(base + kKBytes), kVRow);
        const uint64_t dm = smem_desc_kmajor(smem_u32(sStage + stp * kStageBytes + kKBytes + kVBytes + kOnesBytes), 32);
        const uint32_t sfv_smem = smem_u32(base + kKBytes + kVBytes + kOnesBytes + kMuPad + KB * 512);
#pragma unroll
        for (int t = 0; t < 2; ++t) {
          if (!(ok = warp_wait2(&sh->pc_full[t][j & 1], (j >> 1) & 1, sh, a.status, 23))) break;
          if (elect_one()) {
            tc_fence_after();
            const uint32_t o_col = tmem + O_COL + O_STRIDE * t;
            if constexpr (HYB) {
              if (t == 0) tmem_cp_sf(tmem + SFV_COL, smem_desc_sf_chunk(sfv_smem));
#pragma unroll
              for (int k = 0; k < 4; ++k)                  // 32 keys each; factor byte k of the value rows
                mma_mxf8_ss(o_col, dp[t] + 2 * k, dv + 2 * k, idesc_mxf8_e4m3_e2m1(128, D + 16, k), (j > 0) | (k > 0),
                            tmem + SFP_COL, tmem + SFV_COL);
            } else {
              if (t == 0) {
                tmem_cp_sf(tmem + SFV_COL, smem_desc_sf_chunk(sfv_smem));
                tmem_cp_sf(tmem + SFV_COL + 8, smem_desc_sf_chunk(sfv_smem + 512));
              }
              tmem_cp_sf(tmem + SFP_COL + t * 8, smem_desc_sf_chunk(smem_u32(sSfp + t * kSfpBytes)));
              tmem_cp_sf(tmem + SFP_COL + t * 8 + 4, smem_desc_sf_chunk(smem_u32(sSfp + t * kSfpBytes + 512)));
#pragma unroll
              for (int kb = 0; kb < 2; ++kb)
                mma_nvfp4_ss(o_col, dp[t] + 2 * kb, dv + 2 * kb, idesc_pv, (j > 0) | (kb > 0), tmem + SFP_COL + t * 8 + kb * 4,
                             tmem + SFV_COL + kb * 8);
            }
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
    // my row of the swizzled code tile: 64-byte rows, chunk c sits at chunk position c ^ ((row / 2) % 4)
    // (HYB: 128-byte rows, chunk c at position c ^ (row % 8))
    unsigned char* p_row = sP + t * kPBytes + row * kVRow;
    const int p_xor = (row >> 1) & 3;
    uint32_t* sfp_row = reinterpret_cast<uint32_t*>(sSfp + t * kSfpBytes + (row & 31) * 16 + (row >> 5) * 4);
    const float cs = (a.q_g[bh] * a.k_g[bh]) * a.sl;       // code units -> log2 domain
    float m_run = -INFINITY;
    for (int j = 0; j < nb; ++j) {
      const int ph = j & 1;
      if (!warp_wait2(&sh->s_full[t], ph, sh, a.status, 30)) break;
      tc_fence_after();
      uint32_t s0[32], s1[32], s2[32], s3[32];
      tmem_ld32(lane_base, s0); tmem_ld32(lane_base + 32, s1); tmem_ld32(lane_base + 64, s2); tmem_ld32(lane_base + 96, s3);
      tmem_wait_ld();
      tc_fence_before();
      mbar_arrive(&sh->s_free[t]);                        // the score buffer may be overwritten
      const int nv = a.N - j * 128;                       // >= 128 except on the ragged last tile
      if (nv < 128) {                                     // padded keys: probability zero
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          if (i >= nv) s0[i] = 0xff800000u;
          if (32 + i >= nv) s1[i] = 0xff800000u;
          if (64 + i >= nv) s2[i] = 0xff800000u;
          if (96 + i >= nv) s3[i] = 0xff800000u;
        }
      }
      float mx[8];                                        // maxima of the eight 16-key groups
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
      if constexpr (HYB) {
        // ExpCast-FP8 (Eq. 7): t = (8 u + 120 + beta) / 128, code = round-to-nearest-even(128 t)
        // clipped at 0 (two packed FP32 instructions and a saturating pack per two scores)
        if (j > 0 && !warp_wait2(&sh->o_done[t], (j - 1) & 1, sh, a.status, 31)) break;
        const float fa = cs * 0.0625f, fb = (a.code_off - 8.0f * m_new) * 0.0078125f;
        const uint64_t fa2 = pack_f32x2(fa, fa), fb2 = pack_f32x2(fb, fb);
        auto code4 = [&](const uint32_t (&sv)[32], int w) -> uint32_t {
          return expcast_codes4(sv[4 * w], sv[4 * w + 1], sv[4 * w + 2], sv[4 * w + 3], fa2, fb2);
        };
        auto store16 = [&](const uint32_t (&sv)[32], int half, int chunk) {   // keys 16 chunk .. +15
          const uint4 v = make_uint4(code4(sv, 4 * half), code4(sv, 4 * half + 1), code4(sv, 4 * half + 2), code4(sv, 4 * half + 3));
          *reinterpret_cast<uint4*>(p_row + ((chunk ^ (row & 7)) << 4)) = v;
        };
        store16(s0, 0, 0); store16(s0, 1, 1); store16(s1, 0, 2); store16(s1, 1, 3);
        store16(s2, 0, 4); store16(s2, 1, 5); store16(s3, 0, 6); store16(s3, 1, 7);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");          // my stores -> tensor-core reads
        mbar_arrive(&sh->pc_full[t][j & 1]);
        continue;
      }
      // p = 2^(s cs - m') * 2688: the row maximum maps to 6 * 448, so the largest factor is 448.
      // Per 16-key group: factor = E4M3(max p / 6); element / factor = 2^(s cs + c0 - log2 factor),
      // a zero factor zeroes the group.  The eight factor chains run before the wait below: they
      // do not touch the code tile.
      const float c0 = 11.39231742277876f - m_new;        // log2(2688) - m'
      uint32_t sfw[2] = {0u, 0u};
      float off[8];
#pragma unroll
      for (int g = 0; g < 8; ++g) {
        const float pmax = ex2_approx(fmaf(mx[g], cs, c0));
        const uint32_t sb = (uint32_t)__nv_cvt_float_to_fp8(pmax * (1.0f / 6.0f), __NV_SATFINITE, __NV_E4M3);
        sfw[g >> 2] |= sb << (8 * (g & 3));
        off[g] = sb ? c0 - lg2_approx(decode_ue4m3(sb)) : -INFINITY;
      }
      // the previous code tile must have been consumed before it is overwritten
      if (j > 0 && !warp_wait2(&sh->o_done[t], (j - 1) & 1, sh, a.status, 31)) break;

      const uint64_t cs2 = pack_f32x2(cs, cs);
      auto quant16 = [&](const uint32_t (&sv)[32], int half, int g) -> uint2 {   // keys 16 g .. 16 g + 15
        float v[16];
        const uint64_t off2 = pack_f32x2(off[g], off[g]);
#pragma unroll
        for (int i = 0; i < 16; i += 2) {                 // the exponent's FMA on two scores per instruction
          float x0, x1;
          unpack2(fma2(pack_b32x2(sv[16 * half + i], sv[16 * half + i + 1]), cs2, off2), x0, x1);
          v[i] = ex2_approx(x0);
          v[i + 1] = ex2_approx(x1);
        }
        return make_uint2(cvt_e2m1x8(v[0], v[1], v[2], v[3], v[4], v[5], v[6], v[7]),
                          cvt_e2m1x8(v[8], v[9], v[10], v[11], v[12], v[13], v[14], v[15]));
      };
      auto store32 = [&](const uint32_t (&sv)[32], int chunk) {   // keys 32 chunk .. +31 -> 16 bytes
        const uint2 lo = quant16(sv, 0, 2 * chunk), hi = quant16(sv, 1, 2 * chunk + 1);
        *reinterpret_cast<uint4*>(p_row + ((chunk ^ p_xor) << 4)) = make_uint4(lo.x, lo.y, hi.x, hi.y);
      };
      store32(s0, 0); store32(s1, 1); store32(s2, 2); store32(s3, 3);
      sfp_row[0] = sfw[0];
      sfp_row[128] = sfw[1];                               // the chunk of keys 64..127
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
        const float r_prev = l_now - l_resc;                 // r_{j-1}: sum of the decoded codes
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
        put_pair(r_prev * alpha);
      }
      mbar_arrive(&sh->pc_full[t][j & 1]);
    }
    // ---- last tile's mean term, then the epilogue: O = A / l (means are unscaled at 4 bits, App. B)
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
            __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(r[2 * i]) * inv_l, __uint_as_float(r[2 * i + 1]) * inv_l);
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

template <int D, bool HYB>
cudaError_t run4(const Problem& pr, const QuantLayout& ql, const WorkLayout& wl, const uint8_t* quant,
                 void* o, uint8_t* work, cudaStream_t s) {
  constexpr int KB = D / 64, NVC = HYB ? 1 : 2;
  constexpr size_t kVRow = HYB ? 128 : 64;
  alignas(64) CUtensorMap tq, tk, tv, tmt;
  if (!make_map(&tq, quant + ql.q_codes, D / 2, pr.n_pad, pr.BH, D / 2, 128) ||
      !make_map(&tk, quant + ql.k_codes, D / 2, pr.n_pad, pr.BH, D / 2, 128) ||
      !(HYB ? make_map_u4(&tv, quant + ql.v_codes, (uint64_t)pr.n_pad, D, pr.BH, D)
            : make_map(&tv, quant + ql.v_codes, (uint64_t)pr.n_pad / 2, D, pr.BH, 64, D)) ||
      !make_map(&tmt, work + wl.mu_mma, 32, D, (uint64_t)pr.BH * pr.nb, 32, D))
    return cudaErrorUnknown;
  const size_t n = (size_t)pr.BH * pr.nb * D;
  means_tile_layout_kernel<D><<<(unsigned)((n + 255) / 256), 256, 0, s>>>((const __nv_bfloat16*)(quant + ql.v_means),
                                                                        (float*)(work + wl.mu_mma), n);
  nvfp4_sf_tiles_kernel<D, HYB><<<dim3(pr.nb, pr.BH), 128, 0, s>>>(quant + ql.q_micro, quant + ql.k_micro, quant + ql.v_micro,
                                                                  work + wl.sf_q, work + wl.sf_kv, pr.nb, pr.n_pad);
  Attn4Args a{};
  a.q_g = (const float*)(quant + ql.q_scale);
  a.k_g = (const float*)(quant + ql.k_scale);
  a.sf_q = work + wl.sf_q;
  a.sf_kv = work + wl.sf_kv;
  a.o = (__nv_bfloat16*)o;
  a.status = (uint32_t*)(work + wl.status);
  a.N = pr.N; a.n_pad = pr.n_pad; a.nb = pr.nb;
  a.sl = pr.softmax_scale * 1.4426950408889634f;
  a.code_off = 120.0f + pr.beta;
  a.wait_limit = attn_wait_limit();
  a.wait_hint_ns = attn_wait_hint_ns();
  constexpr size_t stage = 128 * (D / 2) + (D + 16) * kVRow + ((D * 32 + 1023) / 1024) * 1024 + (((KB + NVC) * 512 + 1023) / 1024) * 1024;
  constexpr size_t smem = 1024 + 2 * 128 * (D / 2) + 2 * 128 * kVRow + 2 * 128 * 32 + 2 * 1024 + 2 * 1024 + 1024 + kStages2 * stage + sizeof(FaSmem);
  static_assert(smem <= 227 * 1024, "shared memory of the 4-bit kernel exceeds the SM");
  cudaError_t e = cudaFuncSetAttribute(attn4_fwd_2q_kernel<D, HYB>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  attn4_fwd_2q_kernel<D, HYB><<<dim3((pr.nb + 1) / 2, pr.BH), 640, smem, s>>>(tq, tk, tv, tmt, a);
  count_launches(3);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_attn_fwd4(const Problem& pr, const QuantLayout& ql, const WorkLayout& wl,
                             const uint8_t* quant, void* o, uint8_t* work, cudaStream_t stream) {
  if (hybrid4(pr))
    return pr.d == 128 ? run4<128, true>(pr, ql, wl, quant, o, work, stream) : run4<64, true>(pr, ql, wl, quant, o, work, stream);
  return pr.d == 128 ? run4<128, false>(pr, ql, wl, quant, o, work, stream) : run4<64, false>(pr, ql, wl, quant, o, work, stream);
}

}  // namespace vc
