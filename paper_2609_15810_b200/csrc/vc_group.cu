// Token grouping of VC-Attention for sm_100a (Sec. 3.2 "Value-guided permutation"): for every
// (batch, head) a k-means over the value tokens gives each token a label z_t, and the
// permutation handed to the preprocessing pass is pi = argsort(z), stable, so that every
// cluster becomes one contiguous run of key/value rows (Eq. 3).
//
// The paper fixes neither k nor the initialisation nor the iteration count ("lightweight
// online k-means", warm-started from the previous step's centroids).  This build takes plain
// Lloyd iterations: squared Euclidean distance on the fp32 value rows, centroids started at
// every (N / k)-th token unless warm-started, an empty cluster keeps its centroid, ties go to
// the lower cluster index, and the sort keeps token order inside a cluster.
//
// Everything is deterministic: no floating-point atomics.  A CTA owns a chunk of 1024
// consecutive tokens of one head and forms its per-cluster sums on the tensor core (fixed
// hardware order); a second kernel adds the chunks' partial sums in chunk order.
//
//   group_init_kernel     centroids <- rows 0, N/k, 2 N/k, ...           (cold start only)
//   group_assign_kernel   labels, per-chunk cluster sums and counts      (once per iteration;
//                         distances on the tensor cores, see the kernel)
//   group_update_kernel   centroids <- sum of partial sums / counts      (once per iteration)
//   group_scan_kernel     start of every (cluster, chunk) run in pi
//   group_scatter_kernel  pi: tokens of a chunk in order, behind their cluster's run
#include <cuda_bf16.h>

#include "vc_attn_shared.cuh"
#include "vc_internal.h"
#include "vc_sm100.cuh"

namespace vc {
namespace {

using namespace sm100;

constexpr int kGroupK = 64;          // clusters the kernels are laid out for (k <= 64)
constexpr int kChunkTiles = 8;       // 128-token tiles per chunk
constexpr int kChunk = kChunkTiles * kBlock;

struct GroupArgs {
  const __nv_bfloat16* v;
  int64_t stride_b, stride_h, stride_n;
  int H, N, k, chunks;
  float* centroids;      // [BH][k][D]
  int32_t* labels;       // [BH][N]
  float* psum;           // [BH][chunks][kGroupK][D]
  int32_t* counts;       // [BH][chunks][kGroupK]
  int32_t* offsets;      // [BH][chunks][kGroupK]
  int32_t* perm;         // [BH][N]
  uint32_t* status;      // status word (first word of the workspace)
  uint32_t wait_limit;   // polls after which a wait gives up
  uint32_t nonblocking;  // test hook: polls test the barrier without sleeping in hardware
};

template <int D>
__global__ void group_init_kernel(const GroupArgs a) {
  const int bh = blockIdx.y, j = blockIdx.x, c = threadIdx.x;
  const int b = bh / a.H, h = bh - b * a.H;
  const int step = a.N / a.k > 0 ? a.N / a.k : 1;
  const __nv_bfloat16* row = a.v + b * a.stride_b + h * a.stride_h + (int64_t)(j * step) * a.stride_n;
  if (c < D) a.centroids[((size_t)bh * a.k + j) * D + c] = __bfloat162float(row[c]);
}

// Assignment step on the tensor cores.  The scores v . c of a 128-token tile against the 64
// centroids are a 128 x 64 x d contraction: the value tile arrives by TMA as the bf16 A operand
// (exact: V is bf16), the fp32 centroids are split into three bf16 terms c = c_hi + c_mid + c_lo
// (8 + 8 + 8 mantissa bits, exact), and 3 x d/16 kind::f16 MMAs accumulate every product in FP32
// tensor memory.  label = argmin_c |c|^2 - 2 v.c  (|v|^2 is the same for every c), ties to the
// lower index.  The cluster sums are a contraction too: sums[64 x d] += onehot^T[64 x 128] V[128 x d],
// with the one-hot matrix of the tile's labels written by the token threads (one bf16 1.0 each) and
// the SAME value tile as the B operand, read MN-major (channels contiguous).  Products are exact
// and the accumulation order is the hardware's fixed one: deterministic, no atomics on floats.
//   warp 4      TMA loads of the value tiles (4-stage ring) and MMA issue, one elected lane
//   warps 0-3   one thread per token: scores from tensor memory, argmin, label, one-hot entry
// Tensor memory: two score buffers of 64 columns | cluster sums (d columns, rows = clusters).
constexpr int kGStages = 4;
constexpr uint32_t kGroupWaitLimit = 1u << 22;   // default number of polls of a wait

struct GroupSmem {
  uint64_t v_full[kGStages], v_free[kGStages], s_full[2], s_free[2], oh_full, oh_free;
  uint64_t drain;        // exit: "every MMA of the control warp has completed"
  float cnorm[kGroupK];
  int count_acc[kGroupK];
  uint32_t tmem_base;
  int abort;
  uint32_t wait_limit, nonblocking;
  uint32_t* status;
};

// Bounded wait.  When it gives up, the labels of this chunk are garbage (but in range) and the
// status word says so: vc_poll_status on the workspace returns VC_ERR_TIMEOUT.
__device__ __forceinline__ bool gwait(uint64_t* bar, uint32_t parity, GroupSmem* sh) {
  if (!sh->nonblocking && mbar_try_wait(bar, parity)) return true;
  for (uint32_t i = 0; i < sh->wait_limit; ++i) {
    if (sh->nonblocking ? mbar_test_wait(bar, parity) : mbar_try_wait(bar, parity)) return true;
    if ((i & 255u) == 255u && *reinterpret_cast<volatile int*>(&sh->abort)) return false;
  }
  *reinterpret_cast<volatile int*>(&sh->abort) = 1;
  atomicExch(sh->status, kStatusTimeout | 0x60u);
  return false;
}

__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* m, uint64_t* bar, int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}

// Shared-memory descriptor of an MN-major operand in the 128-byte swizzle: rows of 128 bytes hold
// 64 consecutive M/N elements of one k; 8 k-rows form a 1024-byte group (stride offset), the next
// 64 M/N elements start `mn_block_bytes` further (leading offset).
__device__ __forceinline__ uint64_t smem_desc_mnmajor(uint32_t saddr, uint32_t mn_block_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFF) >> 4);
  d |= (uint64_t)(mn_block_bytes >> 4) << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

template <int D>
__global__ void __launch_bounds__(160, 1) group_assign_kernel(const __grid_constant__ CUtensorMap tm_v, const GroupArgs a) {
  constexpr int KH = D / 64;                        // 128-byte column halves of a bf16 tile
  constexpr uint32_t kVHalf = kBlock * 128, kVStage = KH * kVHalf;       // value tile: [KH][128 tokens][128 B]
  constexpr uint32_t kCHalf = kGroupK * 128, kCSplit = KH * kCHalf;      // centroid term: [KH][64 rows][128 B]
  constexpr uint32_t kOhHalf = 128 * 128;                                // one-hot^T: [2][128 rows][64 tokens]
  constexpr uint32_t SUM_COL = 128;
  constexpr int kTmemCols = 256;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char* sV = smem;                                          // [kGStages] value tiles
  unsigned char* sC = sV + kGStages * kVStage;                       // [3] centroid terms
  unsigned char* sOh = sC + 3 * kCSplit;                             // one-hot^T of the current tile's labels
  GroupSmem* sh = reinterpret_cast<GroupSmem*>(sOh + 2 * kOhHalf);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int chunk = blockIdx.x, bh = blockIdx.y;
  const int b = bh / a.H, h = bh - b * a.H;
  const int tile0 = chunk * kChunkTiles;
  const int n_tiles = min(kChunkTiles, (a.N + kBlock - 1) / kBlock - tile0);

  if (tid == 0) {
    for (int i = 0; i < kGStages; ++i) { mbar_init(&sh->v_full[i], 1); mbar_init(&sh->v_free[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&sh->s_full[i], 1); mbar_init(&sh->s_free[i], 4); }
    mbar_init(&sh->oh_full, 128); mbar_init(&sh->oh_free, 1);
    mbar_init(&sh->drain, 1);
    sh->abort = 0;
    sh->wait_limit = a.wait_limit;
    sh->nonblocking = a.nonblocking;
    sh->status = a.status;
    mbar_fence_init();
    tma_prefetch_desc(&tm_v);
  }
  // centroids -> three bf16 terms in the swizzled K-major operand layout (zero rows beyond k)
  for (int i = tid; i < kGroupK * (D / 8); i += 160) {
    const int j = i / (D / 8), q = i % (D / 8);      // centroid j, channels 8 q .. 8 q + 7
    float c[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) c[e] = j < a.k ? a.centroids[((size_t)bh * a.k + j) * D + 8 * q + e] : 0.f;
    uint32_t w[3][4];
#pragma unroll
    for (int e = 0; e < 8; e += 2) {
      float r0 = c[e], r1 = c[e + 1];
#pragma unroll
      for (int t = 0; t < 3; ++t) {
        const __nv_bfloat162 p2 = __floats2bfloat162_rn(r0, r1);
        w[t][e >> 1] = *reinterpret_cast<const uint32_t*>(&p2);
        r0 -= __low2float(p2);
        r1 -= __high2float(p2);
      }
    }
    const int half = q / 8, chunk16 = q % 8;
    const uint32_t off = half * kCHalf + j * 128 + ((chunk16 ^ (j & 7)) << 4);
#pragma unroll
    for (int t = 0; t < 3; ++t) *reinterpret_cast<uint4*>(sC + t * kCSplit + off) = make_uint4(w[t][0], w[t][1], w[t][2], w[t][3]);
  }
  for (int i = tid; i < 2 * (int)kOhHalf / 16; i += 160) reinterpret_cast<uint4*>(sOh)[i] = make_uint4(0, 0, 0, 0);
  if (tid < kGroupK) {
    float s = INFINITY;                              // an infinite norm keeps the rows beyond k from ever winning
    if (tid < a.k) {
      // all loads first (one dependent global load per channel would cost the whole prologue),
      // then the squares in channel order
      float4 c4[D / 4];
      const float4* src = reinterpret_cast<const float4*>(a.centroids + ((size_t)bh * a.k + tid) * D);
#pragma unroll
      for (int q = 0; q < D / 4; ++q) c4[q] = __ldg(src + q);
      s = 0.f;
#pragma unroll
      for (int q = 0; q < D / 4; ++q) {
        s = fmaf(c4[q].x, c4[q].x, s); s = fmaf(c4[q].y, c4[q].y, s);
        s = fmaf(c4[q].z, c4[q].z, s); s = fmaf(c4[q].w, c4[q].w, s);
      }
    }
    sh->cnorm[tid] = s;
    sh->count_acc[tid] = 0;
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy stores -> tensor-core reads
  if (warp == 4) { tmem_alloc<kTmemCols>(&sh->tmem_base); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sh->tmem_base;

  if (warp == 4) {
    // ------------------------------------------------------------------ loads and MMA issue
    const uint32_t idesc_s = idesc_bf16(128, kGroupK);
    const uint32_t idesc_sum = idesc_bf16(128, D) | (1u << 16);        // B operand MN-major
    int loaded = 0;                                    // value tiles whose copies have been issued
    auto load = [&](int i) {
      const int st = i % kGStages;
      loaded = i + 1;
      if (elect_one()) {
        mbar_expect_tx(&sh->v_full[st], kVStage);
        for (int kh = 0; kh < KH; ++kh)
          tma_load_4d(sV + st * kVStage + kh * kVHalf, &tm_v, &sh->v_full[st], 128 * kh, (tile0 + i) * kBlock, h, b);
      }
      __syncwarp();
    };
    auto scores = [&](int i) -> bool {               // S[i % 2] = V_i C^T, three centroid terms
      const int st = i % kGStages, sb = i & 1;
      if (!__all_sync(0xffffffffu, gwait(&sh->v_full[st], (i / kGStages) & 1, sh))) return false;
      if (i >= 2 && !__all_sync(0xffffffffu, gwait(&sh->s_free[sb], ((i >> 1) - 1) & 1, sh))) return false;
      if (elect_one()) {
        tc_fence_after();
        bool first = true;
        for (int t = 0; t < 3; ++t)
          for (int kh = 0; kh < KH; ++kh) {
            const uint64_t dv = smem_desc_kmajor(smem_u32(sV + st * kVStage + kh * kVHalf), 128);
            const uint64_t dc = smem_desc_kmajor(smem_u32(sC + t * kCSplit + kh * kCHalf), 128);
#pragma unroll
            for (int k = 0; k < 4; ++k) { mma_f16_ss(tmem + 64 * sb, dv + 2 * k, dc + 2 * k, idesc_s, first ? 0u : 1u); first = false; }
          }
        mma_commit(&sh->s_full[sb]);
      }
      __syncwarp();
      return true;
    };
    for (int i = 0; i < kGStages - 1 && i < n_tiles; ++i) load(i);
    bool ok = n_tiles > 0 && scores(0);
    for (int i = 0; ok && i < n_tiles; ++i) {
      const int st = i % kGStages;
      if (i + kGStages - 1 < n_tiles) {              // tile i + 3 goes into the stage tile i - 1 has released
        if (i >= 1 && !(ok = __all_sync(0xffffffffu, gwait(&sh->v_free[(i - 1) % kGStages], ((i - 1) / kGStages) & 1, sh)))) break;
        load(i + kGStages - 1);
      }
      if (i + 1 < n_tiles && !(ok = scores(i + 1))) break;           // scores run one tile ahead of the sums
      if (!(ok = __all_sync(0xffffffffu, gwait(&sh->oh_full, i & 1, sh)))) break;
      if (elect_one()) {
        tc_fence_after();
        // sums += onehot^T (K-major, 128 tokens = two 64-token halves) x V_i (MN-major: 16 tokens = 2048 bytes per step)
        const uint64_t dvb = smem_desc_mnmajor(smem_u32(sV + st * kVStage), kVHalf);
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          const uint64_t doh = smem_desc_kmajor(smem_u32(sOh + half * kOhHalf), 128);
#pragma unroll
          for (int k = 0; k < 4; ++k)
            mma_f16_ss(tmem + SUM_COL, doh + 2 * k, dvb + 128 * (4 * half + k), idesc_sum, (i > 0) | (half > 0) | (k > 0));
        }
        mma_commit(&sh->oh_free);
        mma_commit(&sh->v_free[st]);
      }
      __syncwarp();
    }
    // Nothing this CTA started may outlive it (shared and tensor memory are released at exit, also
    // after a wait gave up): wait for the copies nobody consumed and for the MMAs issued so far.
    for (int jj = loaded > kGStages ? loaded - kGStages : 0; jj < loaded; ++jj)
      mbar_wait(&sh->v_full[jj % kGStages], (jj / kGStages) & 1, 1u << 22);
    if (elect_one()) mma_commit(&sh->drain);
    __syncwarp();
    mbar_wait(&sh->drain, 0, 1u << 22);
  } else {
    // ------------------------------------------------------------------ labels and one-hot entries
    const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);
    // my column of the one-hot^T tile: token tid, 2 bytes inside a 16-byte chunk of row `label`
    const uint32_t oh_col = (tid >> 6) * kOhHalf + (((tid & 63) * 2) & 15);
    const int oh_chunk = ((tid & 63) * 2) >> 4;
    int prev = -1;
    bool alive = true;
    for (int i = 0; i < n_tiles; ++i) {
      const int sb = i & 1;
      const int t0 = (tile0 + i) * kBlock;
      const int n_valid = min(kBlock, a.N - t0);
      if (alive && !gwait(&sh->s_full[sb], (i >> 1) & 1, sh)) alive = false;
      tc_fence_after();
      uint32_t s0[32], s1[32];
      tmem_ld32(lane_base + 64 * sb, s0);
      tmem_ld32(lane_base + 64 * sb + 32, s1);
      tmem_wait_ld();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh->s_free[sb]);
      float best = INFINITY;
      int arg = 0;
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        const float dist = fmaf(-2.0f, __uint_as_float(s0[j]), sh->cnorm[j]);
        if (dist < best) { best = dist; arg = j; }
      }
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        const float dist = fmaf(-2.0f, __uint_as_float(s1[j]), sh->cnorm[32 + j]);
        if (dist < best) { best = dist; arg = 32 + j; }
      }
      const bool valid = tid < n_valid;
      if (valid) {
        a.labels[(size_t)bh * a.N + t0 + tid] = arg;
        atomicAdd(&sh->count_acc[arg], 1);
      }
      // the sums of the previous tile must have read the one-hot tile before it changes
      if (i > 0 && alive && !gwait(&sh->oh_free, (i - 1) & 1, sh)) alive = false;
      if (prev >= 0) *reinterpret_cast<unsigned short*>(sOh + oh_col + prev * 128 + ((oh_chunk ^ (prev & 7)) << 4)) = 0;
      prev = valid ? arg : -1;
      if (valid) *reinterpret_cast<unsigned short*>(sOh + oh_col + arg * 128 + ((oh_chunk ^ (arg & 7)) << 4)) = 0x3f80;   // bf16 1.0
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      mbar_arrive(&sh->oh_full);
    }
    // ---- the chunk's cluster sums: row = cluster (lanes 0..63), d columns
    if (n_tiles > 0 && alive && !gwait(&sh->oh_free, (n_tiles - 1) & 1, sh)) alive = false;
    tc_fence_after();
    const size_t at = (size_t)bh * a.chunks + chunk;
    if (warp < 2) {
      float* dst = a.psum + (at * kGroupK + tid) * D;
#pragma unroll 1
      for (int c = 0; c < D / 32; ++c) {
        uint32_t r[32];
        tmem_ld32(lane_base + SUM_COL + 32 * c, r);
        tmem_wait_ld();
#pragma unroll
        for (int q = 0; q < 8; ++q)
          reinterpret_cast<float4*>(dst + 32 * c)[q] = n_tiles > 0 ? make_float4(__uint_as_float(r[4 * q]), __uint_as_float(r[4 * q + 1]), __uint_as_float(r[4 * q + 2]), __uint_as_float(r[4 * q + 3]))
                                                                      : make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");                // every token's count is in
    if (tid < kGroupK) a.counts[at * kGroupK + tid] = sh->count_acc[tid];
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 4) tmem_dealloc<kTmemCols>(tmem);
}

// centroid <- (sum over chunks, in chunk order) / count; an empty cluster keeps its centroid
template <int D>
__global__ void group_update_kernel(const GroupArgs a) {
  const int bh = blockIdx.y, j = blockIdx.x, c = threadIdx.x;
  if (c >= D) return;
  float s = 0.f;
  int n = 0;
  for (int ch = 0; ch < a.chunks; ++ch) {
    const size_t at = (size_t)bh * a.chunks + ch;
    s += a.psum[(at * kGroupK + j) * D + c];
    n += a.counts[at * kGroupK + j];
  }
  if (n > 0) a.centroids[((size_t)bh * a.k + j) * D + c] = s / (float)n;
}

// offsets[chunk][label] = tokens with a smaller label + tokens of this label in earlier chunks
__global__ void group_scan_kernel(const GroupArgs a) {
  const int bh = blockIdx.x, j = threadIdx.x;   // one thread per label
  __shared__ int total[kGroupK], start[kGroupK];
  int n = 0;
  for (int ch = 0; ch < a.chunks; ++ch) n += a.counts[((size_t)bh * a.chunks + ch) * kGroupK + j];
  total[j] = n;
  __syncthreads();
  if (j == 0) {
    int run = 0;
    for (int l = 0; l < kGroupK; ++l) { start[l] = run; run += total[l]; }
  }
  __syncthreads();
  int run = start[j];
  for (int ch = 0; ch < a.chunks; ++ch) {
    const size_t at = ((size_t)bh * a.chunks + ch) * kGroupK + j;
    a.offsets[at] = run;
    run += a.counts[at];
  }
}

// One warp per chunk walks its tokens in order, 32 at a time: a token goes behind the tokens of
// its label seen so far, and among the 32 of a step behind the lower lanes with the same label.
__global__ void __launch_bounds__(32) group_scatter_kernel(const GroupArgs a) {
  const int chunk = blockIdx.x, bh = blockIdx.y, lane = threadIdx.x;
  __shared__ int next[kGroupK];
  const size_t at = ((size_t)bh * a.chunks + chunk) * kGroupK;
  next[lane] = a.offsets[at + lane];
  next[lane + 32] = a.offsets[at + lane + 32];
  __syncwarp();
  const int t_end = min(a.N, (chunk + 1) * kChunk);
  for (int t0 = chunk * kChunk; t0 < t_end; t0 += 32) {
    const int t = t0 + lane;
    const bool valid = t < t_end;
    const int lab = valid ? a.labels[(size_t)bh * a.N + t] : -1 - lane;   // distinct dummies never match
    const unsigned int same = __match_any_sync(0xffffffffu, lab);
    const int rank = __popc(same & ((1u << lane) - 1u));
    int basepos = 0;
    if (valid) basepos = next[lab];
    __syncwarp();
    if (valid) {
      a.perm[(size_t)bh * a.N + basepos + rank] = t;
      if (rank == __popc(same) - 1) next[lab] = basepos + rank + 1;     // the last of its group moves the cursor
    }
    __syncwarp();
  }
}

// 4-D byte tensor [B][H][N][2 d] with the caller's strides, box {128 bytes, 128 rows}, 128-byte swizzle.
bool make_value_map(CUtensorMap* m, const Problem& pr, const void* v) {
  attn::EncodeTiledFn fn = attn::encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[4] = {(cuuint64_t)pr.d * 2, (cuuint64_t)pr.N, (cuuint64_t)pr.H, (cuuint64_t)pr.B};
  const cuuint64_t strides[3] = {(cuuint64_t)pr.stride_n * 2, (cuuint64_t)pr.stride_h * 2, (cuuint64_t)pr.stride_b * 2};
  const cuuint32_t box[4] = {128, 128, 1, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(v), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D>
cudaError_t run_group(const Problem& pr, GroupArgs a, int iters, int warm, cudaStream_t s) {
  constexpr size_t smem = 1024 + (size_t)kGStages * kBlock * D * 2 + 3 * (size_t)kGroupK * D * 2 + 2 * 128 * 128 + sizeof(GroupSmem);
  alignas(64) CUtensorMap tm_v;
  if (!make_value_map(&tm_v, pr, a.v)) return cudaErrorUnknown;
  cudaError_t e = cudaFuncSetAttribute(group_assign_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  if (!warm) { group_init_kernel<D><<<dim3(a.k, pr.BH), D, 0, s>>>(a); count_launches(1); }
  for (int it = 0; it < iters; ++it) {
    group_assign_kernel<D><<<dim3(a.chunks, pr.BH), 160, smem, s>>>(tm_v, a);
    group_update_kernel<D><<<dim3(a.k, pr.BH), D, 0, s>>>(a);
    count_launches(2);
  }
  group_scan_kernel<<<pr.BH, kGroupK, 0, s>>>(a);
  group_scatter_kernel<<<dim3(a.chunks, pr.BH), 32, 0, s>>>(a);
  count_launches(2);
  return cudaGetLastError();
}

struct GroupLayout {
  size_t status, labels, psum, counts, offsets, total;
  int chunks;
};
GroupLayout group_layout(const Problem& pr) {
  GroupLayout g{};
  g.chunks = (pr.N + kChunk - 1) / kChunk;
  size_t off = 0;
  auto place = [&](size_t bytes) { size_t o = off; off = (off + bytes + 1023) / 1024 * 1024; return o; };
  g.status = place(VC_GROUP_LABELS_OFFSET);          // the status word, then the labels
  g.labels = place((size_t)pr.BH * pr.N * 4);
  g.psum = place((size_t)pr.BH * g.chunks * kGroupK * pr.d * 4);
  g.counts = place((size_t)pr.BH * g.chunks * kGroupK * 4);
  g.offsets = place((size_t)pr.BH * g.chunks * kGroupK * 4);
  g.total = off;
  return g;
}

}  // namespace
}  // namespace vc

using namespace vc;

extern "C" size_t vc_group_workspace_bytes(const vc_params* p) {
  Problem pr;
  if (resolve(p, &pr) != VC_OK) return 0;
  return group_layout(pr).total;
}

extern "C" vc_status vc_group(const vc_params* p, const void* v, int32_t k, int32_t iters, int32_t warm_start,
                              float* centroids, int32_t* perm, void* workspace, void* stream) {
  Problem pr;
  vc_status st = resolve(p, &pr);
  if (st != VC_OK) return st;
  if (!v || !centroids || !perm || !workspace) return VC_ERR_INVALID_ARG;
  if (((uintptr_t)v | (uintptr_t)centroids | (uintptr_t)perm | (uintptr_t)workspace) & 15) return VC_ERR_INVALID_ARG;
  if (k < 1 || iters < 1 || k > pr.N) return VC_ERR_INVALID_ARG;
  if (k > kGroupK) return VC_ERR_UNSUPPORTED;
  const GroupLayout gl = group_layout(pr);
  uint8_t* work = (uint8_t*)workspace;
  GroupArgs a{};
  a.v = (const __nv_bfloat16*)v;
  a.stride_b = pr.stride_b; a.stride_h = pr.stride_h; a.stride_n = pr.stride_n;
  a.H = pr.H; a.N = pr.N; a.k = k; a.chunks = gl.chunks;
  a.centroids = centroids;
  a.labels = (int32_t*)(work + gl.labels);
  a.psum = (float*)(work + gl.psum);
  a.counts = (int32_t*)(work + gl.counts);
  a.offsets = (int32_t*)(work + gl.offsets);
  a.perm = perm;
  a.status = (uint32_t*)(work + gl.status);
  const uint32_t lim = wait_limit_override();
  a.wait_limit = lim ? lim : kGroupWaitLimit;
  a.nonblocking = lim ? 1u : 0u;
  if (cudaMemsetAsync(a.status, 0, 4, (cudaStream_t)stream) != cudaSuccess) return VC_ERR_CUDA;
  const cudaError_t e = pr.d == 128 ? run_group<128>(pr, a, iters, warm_start, (cudaStream_t)stream)
                                    : run_group<64>(pr, a, iters, warm_start, (cudaStream_t)stream);
  return e == cudaSuccess ? VC_OK : VC_ERR_CUDA;
}
