// Internal declarations shared by the translation units of libvc (not part of the ABI).
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "vc_attn.h"

namespace vc {

constexpr int kBlock = 128;   // B_v of Eq. 4 = row block of the Q/K scales = MMA tile

// Resolved parameters: defaults filled in, derived sizes added.
struct Problem {
  int B, H, N, d, BH;
  int grid_t, grid_h, grid_w;
  int bits, p_format, flags;
  float softmax_scale, beta, rope_theta;
  int rope_dim[3];
  int64_t stride_b, stride_h, stride_n;
  int n_pad, nb;
  int heads_per_pass;
  int kernel_variant;
};

// The hybrid 4-bit arrangement: NVFP4 Q^ and K^, ExpCast-FP8 P, E2M1 values under power-of-two
// factors per 32 tokens (the FP8 x FP4 block-scaled product).  Selected by bits = 4 with
// p_format = VC_P_EXPCAST_E4M3.
inline bool hybrid4(const Problem& pr) { return pr.bits == 4 && pr.p_format == VC_P_EXPCAST_E4M3; }

// Byte offsets of the sections of the quantized bundle.
struct QuantLayout {
  size_t q_codes, k_codes, v_codes, q_scale, k_scale, v_scale, v_means, k_mean;
  size_t q_micro, k_micro, v_micro;
  size_t q_codes_bytes, k_codes_bytes, v_codes_bytes, q_scale_bytes, k_scale_bytes,
      v_scale_bytes, v_means_bytes, k_mean_bytes, q_micro_bytes, k_micro_bytes, v_micro_bytes;
  size_t total;
};

// Byte offsets of the sections of the workspace.
struct WorkLayout {
  size_t status;     // uint32 status word (+ padding)
  size_t rope;       // float2 (cos, sin) compact per-axis tables, then the same as (cos + sin, cos - sin)
  size_t k_part;     // fp32 [BH][nb][d] per-block column sums of RoPE(K)
  size_t v_mu;       // fp32 [BH][nb][d] block means of the gathered V
  size_t amax;       // uint32 [BH][d] residual amax bits (8-bit V) then [2][BH] Q/K head amax (4-bit)
  size_t amax_bytes;
  size_t perm_bits;  // uint32 [BH][ceil(N / 32)]: bitmap of the permutation validator (VC_FLAG_CHECK_PERM)
  size_t perm_bits_bytes;
  size_t mu_mma;     // fp32 [BH][nb][d][8]: block means as the B operand of the mean-restoration MMA
  size_t sf_q;       // bytes [BH][nb][d/64][512]: Q^ NVFP4 factors in MMA chunk order (4 bits)
  size_t sf_kv;      // bytes [BH][nb][d/64 + 2][512]: K^ and R^ factors per key tile (4 bits)
  size_t expand;     // bf16 [3][BH][N_pad][d]: NVFP4 operands expanded to bf16, serial 4-bit kernel only
  size_t total;
  int rope_off[3];   // entry offset of each axis table
  int rope_entries;
};

vc_status resolve(const vc_params* p, Problem* out);
QuantLayout quant_layout(const Problem& pr);
WorkLayout work_layout(const Problem& pr);

// Launchers (each returns the CUDA error of its launches; all asynchronous on `stream`).
cudaError_t launch_prep(const Problem& pr, const QuantLayout& ql, const WorkLayout& wl,
                        const void* q, const void* k, const void* v, const int32_t* perm,
                        uint8_t* quant, uint8_t* work, cudaStream_t stream, const vc_prep_stats* stats);
// clear_status: start with a zeroed status word (false inside vc_attn, where the word may already
// hold what the preprocessing pass recorded)
cudaError_t launch_attn_fwd(const Problem& pr, const QuantLayout& ql, const WorkLayout& wl,
                            const uint8_t* quant, void* o, uint8_t* work, cudaStream_t stream, bool clear_status);

cudaError_t launch_attn_fwd4(const Problem& pr, const QuantLayout& ql, const WorkLayout& wl,
                             const uint8_t* quant, void* o, uint8_t* work, cudaStream_t stream);

// Validator of the permutation (VC_FLAG_CHECK_PERM); the status word must have been cleared before.
cudaError_t launch_perm_check(const Problem& pr, const int32_t* perm, const WorkLayout& wl, uint8_t* work, cudaStream_t stream);

void count_launches(int n);

// Status-word codes (first word of a workspace).
constexpr uint32_t kStatusTimeout = 0x100;    // | site code: a bounded device-side wait gave up
constexpr uint32_t kStatusBadPerm = 0x200;    // the permutation validator found a bad entry

// Polls after which a device-side wait gives up (vc_test_set_wait_limit); 0 = the default.
uint32_t wait_limit_override();

}  // namespace vc
