/*
 * vc_attn.h -- C ABI of the VC-Attention hot path on NVIDIA B200 (sm_100a).
 *
 * The library computes low-bit attention for video-diffusion transformers in two stages:
 *
 *   vc_prep      the fused preprocessing pass (paper Sec. 3.4 "Fused preprocessing",
 *                App. B): RoPE, Q/K Hadamard rotation, K channel-mean smoothing, V
 *                per-128-token block-mean smoothing (Eq. 4), gather by the token-group
 *                permutation pi (Eq. 3), padding, quantization to the 8-bit (FP8 E4M3) or
 *                4-bit (NVFP4: E2M1 under a per-16 E4M3 microscale) formats with scales.
 *   vc_attn_fwd  the quantized attention forward: low-bit Q K^T, the online softmax of
 *                Eq. 1 whose exponent is written directly as an E4M3 probability code
 *                (ExpCast-FP8, Eq. 7), low-bit P V, and the block means added back inside
 *                the recurrence (Eq. 6); epilogue O = s_V * A / l.
 *   vc_attn      vc_prep followed by vc_attn_fwd.
 *   vc_group     the producer of the token-group permutation pi (Sec. 3.2): k-means on V,
 *                stable argsort of the labels.
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer unless the name says host; all must be 16-byte
 *     aligned.  The caller owns every buffer; the library allocates no device memory.
 *   - All work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = the legacy
 *     default stream).  No entry point synchronizes except vc_poll_status and
 *     vc_attn_host.
 *   - Errors are return codes only.  Argument errors are detected on the host before any
 *     launch.  A device-side wait that exceeds its spin limit writes a code to the status
 *     word at the start of the workspace and the kernel exits normally; vc_poll_status
 *     reads it back as VC_ERR_TIMEOUT.
 *   - Q, K, V are [B, H, N, d] bf16 with d contiguous; strides are given in elements
 *     (0 = packed).  N tokens form a T x Hg x Wg grid in row-major (t, y, x) order.
 *     O is [B, H, N, d] bf16, packed, in the original query order.
 */
#ifndef VC_ATTN_H_
#define VC_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  VC_OK = 0,
  VC_ERR_INVALID_ARG = 1,   /* null pointer, bad size, misaligned pointer; from
                               vc_poll_status: `perm` was not a permutation          */
  VC_ERR_UNSUPPORTED = 2,   /* a combination this build does not implement           */
  VC_ERR_WORKSPACE = 3,     /* reserved                                              */
  VC_ERR_CUDA = 4,          /* a CUDA runtime/driver call failed                     */
  VC_ERR_TIMEOUT = 5,       /* a bounded device-side wait gave up                    */
  VC_ERR_SCRATCH_LIMIT = 6  /* vc_prep_noalloc: the problem needs more scratch than
                               VC_NOALLOC_SCRATCH_BYTES                              */
} vc_status;

/* probability formats of the softmax stage (Sec. 3.3, App. A "Scope of ExpCast-FP8") */
enum {
  VC_P_DEFAULT = 0,         /* ExpCast-FP8 at 8 bits, NVFP4 at 4 bits                */
  /* Eq. 7: one FMA, the byte viewed as E4M3.  With bits = 4 this selects the HYBRID 4-bit
   * arrangement: Q^ and K^ stay NVFP4, P is the ExpCast-FP8 code, and the value residual is
   * stored as E2M1 under one power-of-two factor (an exponent byte, value 2^(byte - 127)) per
   * channel and 32 consecutive permuted tokens, so that the value product runs as an
   * FP8 x FP4 block-scaled MMA.  The factor is the smallest power of two that keeps the
   * group's maximum inside the E2M1 range (no clipping); a group of zeros stores byte 0.
   * vc_attn_fwd then wants the bundle 32-byte aligned; kernel_variant must be 0.            */
  VC_P_EXPCAST_E4M3 = 1,
  VC_P_EXP_E4M3 = 2,        /* exponentiate, then cast to E4M3 (Fig. 4a upper box)   */
  VC_P_NVFP4 = 3,           /* E2M1 under a per-16-key E4M3 microscale               */
  /* the same result as VC_P_EXP_E4M3 up to the polynomial's error (relative 3.7e-6, so a code
   * differs from the exactly exponentiated one for about one score in 10^4): 2^u evaluated on
   * the FMA pipe by a degree-4 polynomial instead of the special-function unit, for every
   * score (POLY) or for one score in four (MIX).  They exist to measure where the exponential
   * belongs on this GPU (Sec. 3.3); kernel_variant 1 computes them like VC_P_EXP_E4M3.        */
  VC_P_EXP_POLY_E4M3 = 4,
  VC_P_EXP_MIX_E4M3 = 5
};

/* stages of the chain that can be switched off (all on = the paper's method) */
enum {
  VC_FLAG_ROPE = 1,
  VC_FLAG_HADAMARD = 2,
  VC_FLAG_K_SMOOTH = 4,
  VC_FLAG_V_SMOOTH = 8,
  VC_FLAG_ALL = 15,
  /* variant switch, not part of VC_FLAG_ALL: 8-bit Q^ and K^ as INT8 (symmetric, scale amax/127
   * per 128 rows) and Q^ K^T as an integer product -- the arrangement the paper runs on B200
   * (Fig. 3); default is FP8 E4M3 for both products (the paper's B300 arrangement, Sec. 4.5).
   * bits = 8 and the pipelined kernel only. */
  VC_FLAG_INT8_QK = 16,
  /* check switch, not part of VC_FLAG_ALL: vc_prep also runs a validator over `perm` (Eq. 3
   * needs a permutation of [0, N) per head).  An entry outside [0, N) or one that occurs twice
   * is recorded in the status word and vc_poll_status returns VC_ERR_INVALID_ARG.  With or
   * without this flag the gather itself clamps every entry into [0, N), so a bad `perm` gives a
   * wrong bundle, never an out-of-bounds read. */
  VC_FLAG_CHECK_PERM = 32
};

typedef struct {
  int32_t B, H, N, d;               /* d in {64, 128}; 1 <= N <= 2^22; B * H <= 65535   */
  int32_t grid_t, grid_h, grid_w;   /* grid_t * grid_h * grid_w == N                    */
  int32_t bits;                     /* 8 or 4                                           */
  int32_t p_format;                 /* VC_P_*                                           */
  int32_t flags;                    /* VC_FLAG_*                                        */
  float softmax_scale;              /* 0 => 1/sqrt(d)                                   */
  float beta;                       /* ExpCast offset of Eq. 7; 0 => -0.35              */
  int32_t rope_dim_t, rope_dim_h, rope_dim_w; /* channels per axis, even, sum == d;
                                       all 0 => (d - 4*(d/6), 2*(d/6), 2*(d/6))         */
  float rope_theta;                 /* 0 => 10000                                       */
  int64_t stride_b, stride_h, stride_n;       /* of Q, K and V, in elements; 0 => packed; stride_n < 2^30 */
  int32_t heads_per_pass;           /* heads preprocessed per launch group (L2 reuse of
                                       the second read of K and V); 0 => library default */
  int32_t kernel_variant;           /* attention kernel: 0 = pipelined, two query tiles per
                                       CTA (default); 1 = simple serial kernel, kept for
                                       A/B measurement and cross-checks                  */
  int32_t block_q, block_k, block_v; /* rows per Q and per K scale block, tokens per value
                                       block B_v of Eq. 4 (Sec. 3.2 "Block demeaning").  0 =>
                                       128.  The kernels are laid out for 128 (one block = one
                                       MMA tile, so a scale folds into the softmax constant and
                                       a block mean into one rank-one update per tile); any
                                       other value returns VC_ERR_UNSUPPORTED              */
} vc_params;

/* Device pointers into the quantized bundle written by vc_prep (N_pad = 128*ceil(N/128),
 * nb = N_pad/128, BH = B*H).  8 bits: codes are E4M3 bytes (Q^, K^: two's-complement INT8
 * bytes under VC_FLAG_INT8_QK).  4 bits: codes are E2M1
 * nibbles, two per byte, the even index in the low nibble; micro are unsigned E4M3 bytes.
 *   q_codes [BH][N_pad][d]      (4 bits: [BH][N_pad][d/2])   rows in query order
 *   k_codes [BH][N_pad][d]      (4 bits: [BH][N_pad][d/2])   rows in permuted order
 *   v_codes [BH][d][N_pad]      (4 bits: [BH][d][N_pad/2])   residual, channel-major
 *   q_scale [BH][nb] fp32       (4 bits: [BH], the outer NVFP4 scale g_Q)
 *   k_scale [BH][nb] fp32       (4 bits: [BH], g_K)
 *   v_scale [BH][d]  fp32       (4 bits: all ones)
 *   v_means [BH][nb][d] bf16    block means / v_scale (4 bits: unscaled), App. B
 *   k_mean  [BH][d]  fp32       post-RoPE channel mean of K
 *   q_micro [BH][N_pad][d/16], k_micro [BH][N_pad][d/16], v_micro [BH][d][N_pad/16]  (4 bits)
 * Hybrid 4-bit arrangement (bits = 4, p_format = VC_P_EXPCAST_E4M3): as at 4 bits, except
 *   v_micro [BH][d][N_pad/32]   exponent bytes of the power-of-two factors, 32 tokens each
 */
typedef struct {
  void *q_codes, *k_codes, *v_codes;
  float *q_scale, *k_scale, *v_scale;
  void *v_means;
  float *k_mean;
  void *q_micro, *k_micro, *v_micro;
  size_t q_codes_bytes, k_codes_bytes, v_codes_bytes, q_scale_bytes, k_scale_bytes,
         v_scale_bytes, v_means_bytes, k_mean_bytes, q_micro_bytes, k_micro_bytes,
         v_micro_bytes;
} vc_quant_ptrs;

/* Sizes (bytes) of the caller-allocated quantized bundle and workspace; 0 on bad params. */
size_t vc_quant_bytes(const vc_params *p);
size_t vc_workspace_bytes(const vc_params *p);

/* Preprocessing pass (Sec. 3.4, App. B).  perm: int32 [B][H][N], row t of the permuted
 * K/V is row perm[t] of the input (Eq. 3), or NULL for the identity; it must be a
 * permutation of [0, N) per (b, h).  Entries are clamped into [0, N) before they are used
 * as row indices; VC_FLAG_CHECK_PERM adds a validator that reports a bad entry through the
 * status word.  Writes `quant`; uses `workspace` (contents on entry irrelevant; the first 4
 * bytes become the status word). */
vc_status vc_prep(const vc_params *p, const void *q, const void *k, const void *v,
                  const int32_t *perm, void *quant, void *workspace, void *stream);

/* The statistics of the pass: what makes it read K and V twice.  App. B has the K pass fuse "the
 * centering statistics" and the V pass "the block mean and scale reductions"; a caller whose
 * producer of K and V (the projection in front of attention) already has them can hand them in,
 * and the pass then runs without its statistics launches: K and V are read once.
 *   k_mean        [B*H][d]      fp32  channel mean over all N tokens of K AFTER RoPE (Sec. 3.4)
 *   v_block_mean  [B*H][nb][d]  fp32  mean of every 128-token block of the PERMUTED V (Eq. 4; the
 *                                     ragged last block over its valid tokens; zeros with V smoothing off)
 *   v_amax        [B*H][d]      fp32  max |V' - block mean| per channel over all tokens, >= 0
 * All device pointers, 16-byte aligned.  8 bits only (VC_ERR_UNSUPPORTED at 4 bits, where the
 * outer scales of Q and K are whole-head statistics as well).  The bundle is the one vc_prep
 * writes when the statistics are the ones it would have computed; v_amax may be any upper
 * bound of the true maximum at the price of coarser value codes. */
typedef struct {
  const float *k_mean, *v_block_mean, *v_amax;
} vc_prep_stats;
vc_status vc_prep_with_stats(const vc_params *p, const void *q, const void *k, const void *v,
                             const int32_t *perm, const vc_prep_stats *stats, void *quant,
                             void *workspace, void *stream);
/* Where the last vc_prep call with this bundle and workspace left its own statistics (8 bits);
 * valid until the workspace is used again. */
vc_status vc_prep_stats_view(const vc_params *p, const void *quant, const void *workspace,
                             vc_prep_stats *out);

/* Quantized attention forward (Eq. 1, Eq. 6, Eq. 7) from a bundle in vc_prep's layout.
 * o: [B][H][N][d] bf16.  workspace as above.  `p` must describe the bundle: the same shape,
 * bits, p_format (it selects the value format at 4 bits) and flags as the vc_prep call that
 * wrote it, and `quant` must hold vc_quant_bytes(p) bytes; a mismatch is not detected. */
vc_status vc_attn_fwd(const vc_params *p, const void *quant, void *o, void *workspace,
                      void *stream);

/* vc_prep followed by vc_attn_fwd on the same stream. */
vc_status vc_attn(const vc_params *p, const void *q, const void *k, const void *v,
                  const int32_t *perm, void *o, void *quant, void *workspace, void *stream);

/* The same with HOST input/output buffers (pinned memory recommended): copies q, k, v
 * (packed [B][H][N][d] bf16) and perm (or NULL) to the device staging buffers q_dev,
 * k_dev, v_dev, perm_dev, runs vc_attn, copies o_dev to o_host and synchronizes the
 * stream.  The staging buffers are caller-allocated device memory of the same sizes.
 * Heads are independent, so the call works through groups of heads and overlaps the
 * input copy of the next group and the output copy of the previous one with the kernels of
 * the current one, on two helper streams of its own (made on the first call on a device and kept;
 * calls on one device take turns; ordered after the work already on `stream`; `stream` is
 * complete when the call returns). */
vc_status vc_attn_host(const vc_params *p, const void *q_host, const void *k_host,
                       const void *v_host, const int32_t *perm_host, void *o_host,
                       void *q_dev, void *k_dev, void *v_dev, int32_t *perm_dev, void *o_dev,
                       void *quant, void *workspace, void *stream);

/* Token grouping (Sec. 3.2 "Value-guided permutation"): per (b, h) a k-means over the value
 * tokens labels every token, and perm = argsort(labels), stable: row t of the permuted K/V is
 * row perm[t] of the input (Eq. 3), every cluster one contiguous run.  The output is the `perm`
 * argument of vc_prep / vc_attn; a caller following the paper's schedule (Sec. 3.4 "Amortized
 * grouping schedule") calls this on the first ceil(n/4) denoising steps, every 4th step, with
 * warm_start = 1 after the first call, and reuses `perm` in between.
 *   v          [B][H][N][d] bf16, strides as in vc_params
 *   k          clusters, 1 <= k <= min(N, 64)
 *   iters      Lloyd iterations (assign, then update), >= 1; labels are those of the last assignment
 *   warm_start 0: centroids start at rows 0, N/k, 2 N/k, ... of V; 1: at the values in `centroids`
 *   centroids  [B][H][k][d] fp32, in (warm start) and out (after the last update)
 *   perm       out, int32 [B][H][N]
 *   workspace  vc_group_workspace_bytes(p) bytes; its first 4 bytes are the status word
 *              (vc_poll_status(workspace, stream) reports a device-side wait that gave up as
 *              VC_ERR_TIMEOUT; `perm` is then not valid), and on return the B*H*N int32 at byte
 *              offset VC_GROUP_LABELS_OFFSET are the labels
 * The paper leaves k, the initialisation and the iteration count open; distances are squared
 * Euclidean on the fp32 rows, ties go to the lower cluster index, an empty cluster keeps its
 * centroid.  Deterministic (no floating-point atomics).  Returns VC_ERR_UNSUPPORTED for k > 64. */
#define VC_GROUP_LABELS_OFFSET 1024
size_t vc_group_workspace_bytes(const vc_params *p);
vc_status vc_group(const vc_params *p, const void *v, int32_t k, int32_t iters, int32_t warm_start,
                   float *centroids, int32_t *perm, void *workspace, void *stream);

/* Amortized grouping schedule (Sec. 3.4 "Amortized grouping schedule", App. A "Grouping
 * schedule"): host logic keyed on the denoising step index alone.  Value grouping and demeaning
 * run on the first ceil(n_steps / 4) steps; inside that window the permutation is recomputed on
 * every `reuse`-th step (the paper uses 4) and reused in between; the remaining steps run the
 * plain low-bit kernel on the permutation the window left behind.
 *   VC_GROUP_RECOMPUTE  call vc_group (warm-started after step 0), then vc_attn with V smoothing
 *   VC_GROUP_REUSE      vc_attn with V smoothing and the permutation at hand
 *   VC_GROUP_FROZEN     past the window: the permutation at hand, flags without VC_FLAG_V_SMOOTH
 * Returns -1 for step < 0, step >= n_steps or reuse < 1. */
enum { VC_GROUP_RECOMPUTE = 0, VC_GROUP_REUSE = 1, VC_GROUP_FROZEN = 2 };
int32_t vc_group_schedule(int32_t step, int32_t n_steps, int32_t reuse);

/* vc_prep without a workspace argument and without any allocation.  (The paper has no
 * counterpart: this entry point exists for the sake of its callers, not of the method.)
 *
 * Who needs it: code that runs where device memory may not be requested -- inside a
 * framework that hands a plug-in a fixed set of buffers and forbids it to grow them, in a
 * serving loop that has frozen its memory map after start-up, or on a thread that must not
 * take the driver's allocation lock (cudaMalloc synchronizes the whole device).  Such a
 * caller still owns q, k, v, perm and the output bundle `quant`, but has nowhere to put
 * the pass's scratch.
 *
 * The scratch therefore lives inside the library, in one fixed array of
 * VC_NOALLOC_SCRATCH_BYTES in device global memory.  Every GPU on which the library is
 * used holds that array until the process exits.  Consequences:
 *   - Problems whose scratch need exceeds the limit are refused with VC_ERR_SCRATCH_LIMIT
 *     before anything is launched.  The need is 8 bytes per RoPE table entry plus about
 *     8 * B*H * ceil(N/128) * d bytes (e.g. B*H = 12, N = 32760, d = 128 needs 3.2 MB).
 *   - All calls on a device share the array, and it keeps whatever the previous call left
 *     in it.  The call itself clears the words that have to start at zero, on `stream`.
 *     Two calls that overlap on the GPU (different streams, or different host threads
 *     without ordering between their streams) race on the array: serialize them.
 *   - The first call on each device looks up the array's device address
 *     (cudaGetSymbolAddress) with that device current; make that first call outside any
 *     stream capture.  Later calls only set the kernels' shared-memory attribute (a host-side
 *     call that allocates nothing), launch kernels and issue two small memsets on `stream`.
 * It calls no cudaMalloc / cudaFree and no allocating library routine.  The output is
 * the same bundle vc_prep writes. */
#define VC_NOALLOC_SCRATCH_BYTES (4u << 20)
vc_status vc_prep_noalloc(const vc_params *p, const void *q, const void *k, const void *v,
                          const int32_t *perm, void *quant, void *stream);

/* Device pointers of the bundle's sections (for tests and for feeding a bundle in). */
vc_status vc_quant_view(const vc_params *p, const void *quant, vc_quant_ptrs *out);

/* Synchronizes `stream` and returns VC_ERR_TIMEOUT if a kernel recorded a timed-out wait,
 * VC_ERR_INVALID_ARG if the validator of VC_FLAG_CHECK_PERM found `perm` not to be a
 * permutation, VC_ERR_CUDA on a CUDA error, VC_OK otherwise.  Clears the status word.
 * `workspace` is the workspace of vc_prep / vc_attn_fwd / vc_attn or that of vc_group. */
vc_status vc_poll_status(void *workspace, void *stream);

/* Test hook: the number of polls after which a device-side wait gives up (every mbarrier wait
 * of the attention kernels, the per-head waits of the preprocessing pass, the waits of the
 * grouping kernel).  0 restores the default (about one second).  A tiny value makes waits run
 * out on a correct run, which is how the time-out path is exercised without hanging anything:
 * the kernels then record VC_ERR_TIMEOUT, drain their own copies in flight, free their tensor
 * memory and return; outputs of such a call are invalid.  Process-wide; not for production. */
void vc_test_set_wait_limit(uint32_t polls);

/* Test hook: the ExpCast-FP8 probability code (Eq. 7) formed exactly as the softmax stage of the
 * attention kernels forms it, on its own.  codes[i] is the E4M3 byte of score s[i] (FP32, in units
 * of the integer-like score product) under the factor `cs` that takes such units to the log2
 * domain (> 0) and the running row maximum `m` (log2 domain; s[i] * cs <= m is the caller's
 * business): round-to-nearest-even(8 (s cs - m) + 120 + beta), clipped at 0.  beta 0 => -0.35.
 * `s` and `codes` are device pointers, 16-byte aligned; n is a multiple of 4.  Asynchronous on
 * `stream`; VC_ERR_INVALID_ARG for a bad argument.  Not for production. */
vc_status vc_test_expcast_codes(const float *s, int64_t n, float cs, float m, float beta,
                                uint8_t *codes, void *stream);

/* Measurement aid (Sec. 3.1 "The softmax bottleneck" compares the softmax stage with the time of
 * the two matrix products): the rate at which this GPU executes the products' MMAs with
 * everything else taken away.  Every SM issues `groups` back-to-back 128 x 128 x 128 products of
 * one kind on tiles resident in shared memory, accumulators in tensor memory:
 *   kind 8   tcgen05.mma kind::f8f6f4, E4M3 x E4M3               (the 8-bit products)
 *   kind 4   tcgen05.mma kind::mxf4nvf4.block_scale.block16      (the NVFP4 products)
 * scratch: 8 bytes of device memory, 8-byte aligned.  tflops (host): 2 x MACs of all SMs / the
 * launch's CUDA-event time; mac_per_clk_sm (host): MACs of one SM / its own cycle count.
 * Synchronizes `stream`.  VC_ERR_TIMEOUT if the bounded wait for the MMAs gave up. */
vc_status vc_mma_peak(int32_t kind, int32_t groups, void *scratch, double *tflops, double *mac_per_clk_sm,
                      void *stream);

/* Number of kernels this library has launched in this process (diagnostics). */
uint64_t vc_launch_count(void);

const char *vc_status_string(vc_status s);

#ifdef __cplusplus
}
#endif
#endif /* VC_ATTN_H_ */
