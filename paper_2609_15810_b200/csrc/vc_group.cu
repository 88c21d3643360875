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
// consecutive tokens of one head, adds up its members per cluster in a fixed order, and a
// second kernel adds the chunks' partial sums in chunk order.
//
//   group_init_kernel     centroids <- rows 0, N/k, 2 N/k, ...           (cold start only)
//   group_assign_kernel   labels, per-chunk cluster sums and counts      (once per iteration)
//   group_update_kernel   centroids <- sum of partial sums / counts      (once per iteration)
//   group_scan_kernel     start of every (cluster, chunk) run in pi
//   group_scatter_kernel  pi: tokens of a chunk in order, behind their cluster's run
#include <cuda_bf16.h>

#include "vc_internal.h"

namespace vc {
namespace {

constexpr int kGroupK = 64;          // clusters the kernels are laid out for (k <= 64)
constexpr int kChunkTiles = 8;       // 128-token tiles per chunk
constexpr int kChunk = kChunkTiles * kBlock;
constexpr int kGThreads = 256;

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
};

template <int D>
__global__ void group_init_kernel(const GroupArgs a) {
  const int bh = blockIdx.y, j = blockIdx.x, c = threadIdx.x;
  const int b = bh / a.H, h = bh - b * a.H;
  const int step = a.N / a.k > 0 ? a.N / a.k : 1;
  const __nv_bfloat16* row = a.v + b * a.stride_b + h * a.stride_h + (int64_t)(j * step) * a.stride_n;
  if (c < D) a.centroids[((size_t)bh * a.k + j) * D + c] = __bfloat162float(row[c]);
}

// Shared memory: V tile [128][2 D + 16 B] | centroids [64][4 D + 16 B] | psum [64][D] fp32 |
// cnorm [64] | labels [128] | counts [64].
template <int D>
__global__ void __launch_bounds__(kGThreads, 2) group_assign_kernel(const GroupArgs a) {
  constexpr int VP = 2 * D + 16, CP = 4 * D + 16;
  extern __shared__ __align__(16) unsigned char smem[];
  unsigned char* sV = smem;
  unsigned char* sC = sV + kBlock * VP;
  float* sSum = reinterpret_cast<float*>(sC + kGroupK * CP);
  float* sNorm = sSum + kGroupK * D;
  int* sLab = reinterpret_cast<int*>(sNorm + kGroupK);
  int* sCnt = sLab + kBlock;

  const int tid = threadIdx.x, chunk = blockIdx.x, bh = blockIdx.y;
  const int b = bh / a.H, h = bh - b * a.H;
  const __nv_bfloat16* base = a.v + b * a.stride_b + h * a.stride_h;

  // centroids (zero rows beyond k, which an infinite norm keeps from ever winning)
  for (int i = tid; i < kGroupK * (D / 4); i += kGThreads) {
    const int j = i / (D / 4), q = i % (D / 4);
    float4 c4 = make_float4(0.f, 0.f, 0.f, 0.f);
    if (j < a.k) c4 = *reinterpret_cast<const float4*>(a.centroids + ((size_t)bh * a.k + j) * D + 4 * q);
    *reinterpret_cast<float4*>(sC + j * CP + 16 * q) = c4;
  }
  for (int i = tid; i < kGroupK * D; i += kGThreads) sSum[i] = 0.f;
  if (tid < kGroupK) sCnt[tid] = 0;
  __syncthreads();
  if (tid < kGroupK) {
    float s = INFINITY;
    if (tid < a.k) {
      s = 0.f;
      for (int c = 0; c < D; ++c) {
        const float x = *reinterpret_cast<const float*>(sC + tid * CP + 4 * c);
        s = fmaf(x, x, s);
      }
    }
    sNorm[tid] = s;
  }

  // 4 tokens x 8 centroids per thread: tokens tg, tg + 32, ... and centroids cg, cg + 8, ..., so that
  // the lanes of a warp read consecutive (padded) rows of either tile: no bank conflicts
  const int tg = tid >> 3, cg = tid & 7;
  for (int tile = 0; tile < kChunkTiles; ++tile) {
    const int t0 = chunk * kChunk + tile * kBlock;
    if (t0 >= a.N) break;
    __syncthreads();                         // the previous tile's readers are done with sV / sLab
    for (int i = tid; i < kBlock * (D / 8); i += kGThreads) {
      const int row = i / (D / 8), q = i % (D / 8);
      uint4 val = make_uint4(0, 0, 0, 0);
      if (t0 + row < a.N) val = __ldg(reinterpret_cast<const uint4*>(base + (int64_t)(t0 + row) * a.stride_n + 8 * q));
      *reinterpret_cast<uint4*>(sV + row * VP + 16 * q) = val;
    }
    __syncthreads();

    // scores[token][centroid] = v . c
    float acc[4][8];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;
#pragma unroll 2
    for (int d8 = 0; d8 < D / 8; ++d8) {
      float vv[4][8];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint4 raw = *reinterpret_cast<const uint4*>(sV + (tg + 32 * i) * VP + 16 * d8);
        const unsigned int w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          vv[i][2 * q] = __uint_as_float(w[q] << 16);
          vv[i][2 * q + 1] = __uint_as_float(w[q] & 0xffff0000u);
        }
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const float4 c0 = *reinterpret_cast<const float4*>(sC + (cg + 8 * j) * CP + 32 * d8);
        const float4 c1 = *reinterpret_cast<const float4*>(sC + (cg + 8 * j) * CP + 32 * d8 + 16);
        const float cc[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int e = 0; e < 8; ++e) acc[i][j] = fmaf(vv[i][e], cc[e], acc[i][j]);
      }
    }
    // label = argmin_c |c|^2 - 2 v.c  (|v|^2 is the same for every c); ties -> lower index
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float best = INFINITY;
      int arg = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const float dist = fmaf(-2.0f, acc[i][j], sNorm[cg + 8 * j]);
        if (dist < best) { best = dist; arg = cg + 8 * j; }
      }
#pragma unroll
      for (int s = 1; s < 8; s <<= 1) {
        const float ob = __shfl_xor_sync(0xffffffffu, best, s);
        const int oa = __shfl_xor_sync(0xffffffffu, arg, s);
        if (ob < best || (ob == best && oa < arg)) { best = ob; arg = oa; }
      }
      if (cg == 0) sLab[tg + 32 * i] = arg;
    }
    __syncthreads();
    if (tid < kBlock && t0 + tid < a.N) a.labels[(size_t)bh * a.N + t0 + tid] = sLab[tid];
    // cluster sums of the tile, column c by thread c, tokens in order: a fixed summation order
    if (tid < D) {
      const int n_valid = min(kBlock, a.N - t0);
      for (int t = 0; t < n_valid; ++t) {
        const float x = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(sV + t * VP + 2 * tid));
        sSum[sLab[t] * D + tid] += x;
      }
    } else if (tid == D) {
      const int n_valid = min(kBlock, a.N - t0);
      for (int t = 0; t < n_valid; ++t) sCnt[sLab[t]] += 1;
    }
  }
  __syncthreads();
  const size_t at = (size_t)bh * a.chunks + chunk;
  for (int i = tid; i < kGroupK * D; i += kGThreads) a.psum[at * kGroupK * D + i] = sSum[i];
  if (tid < kGroupK) a.counts[at * kGroupK + tid] = sCnt[tid];
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

template <int D>
cudaError_t run_group(const Problem& pr, GroupArgs a, int iters, int warm, cudaStream_t s) {
  constexpr size_t smem = (size_t)kBlock * (2 * D + 16) + (size_t)kGroupK * (4 * D + 16) + (size_t)kGroupK * D * 4 +
                          kGroupK * 4 + kBlock * 4 + kGroupK * 4;
  cudaError_t e = cudaFuncSetAttribute(group_assign_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  if (!warm) { group_init_kernel<D><<<dim3(a.k, pr.BH), D, 0, s>>>(a); count_launches(1); }
  for (int it = 0; it < iters; ++it) {
    group_assign_kernel<D><<<dim3(a.chunks, pr.BH), kGThreads, smem, s>>>(a);
    group_update_kernel<D><<<dim3(a.k, pr.BH), D, 0, s>>>(a);
    count_launches(2);
  }
  group_scan_kernel<<<pr.BH, kGroupK, 0, s>>>(a);
  group_scatter_kernel<<<dim3(a.chunks, pr.BH), 32, 0, s>>>(a);
  count_launches(2);
  return cudaGetLastError();
}

struct GroupLayout {
  size_t labels, psum, counts, offsets, total;
  int chunks;
};
GroupLayout group_layout(const Problem& pr) {
  GroupLayout g{};
  g.chunks = (pr.N + kChunk - 1) / kChunk;
  size_t off = 0;
  auto place = [&](size_t bytes) { size_t o = off; off = (off + bytes + 1023) / 1024 * 1024; return o; };
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
  const cudaError_t e = pr.d == 128 ? run_group<128>(pr, a, iters, warm_start, (cudaStream_t)stream)
                                    : run_group<64>(pr, a, iters, warm_start, (cudaStream_t)stream);
  return e == cudaSuccess ? VC_OK : VC_ERR_CUDA;
}
