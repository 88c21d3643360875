// Fused 8-bit preprocessing pass of VC-Attention for sm_100a (Sec. 3.4 "Fused preprocessing",
// App. B): ONE persistent launch that reads Q, K, V as bf16 and writes codes, scales and block
// means; no rotated / permuted / centered high-precision tensor reaches HBM.
//
// The pass has two global reductions per head (the channel mean of RoPE(K) over all tokens, and
// the per-channel maximum of the V residual over all tokens, which sets the value scale), so K
// and V are touched twice.  Both touches happen inside this launch, close enough in time that
// the second one is served from L2:
//
//   work items, 128 rows (tokens) each        what they do
//   KS(h, blk)  K statistics                  column sums of RoPE(K) of the block
//   VS(h, blk)  V statistics                  gather by pi; block mean (Eq. 4), max and min per channel
//   QQ(h, blk)  Q quantization                RoPE, Hadamard, per-block scale, codes
//   KQ(h, blk)  K quantization                gather, RoPE at the source position, - mean, Hadamard, scale, codes
//   VQ(h, blk)  V quantization                gather, residual, per-channel scale, codes channel-major, means
//
// Items are numbered head by head: [KS, VS of every block, ascending] [QQ of every block]
// [KQ, VQ of every block, DESCENDING], so that the quantizing items re-read the blocks the
// statistics items touched last first, and the Q items of the head separate the two phases.
// A CTA is three independent workers (warpgroups of 128 threads, named barriers); worker w of
// all takes items w, w + W, w + 2 W, ...  The last statistics item of a head to finish (a
// counter in the workspace) folds the partial sums into the head's mean and scales and raises
// the head's ready flag; a quantizing item of K or V polls that flag first, with a bounded
// spin that records a time-out in the status word instead of hanging.  Every item with a
// smaller number than a waiting item is owned by a running worker that waits for nothing but
// items smaller still, so the wait always ends (the grid never exceeds one CTA per SM).
//
// Per item the 16-byte chunks of the NEXT item are on their way into the other shared-memory
// stage (cp.async, zero-fill for padding rows) while the current one is transformed.
//
// Arithmetic of the row items, one row per thread with all d channels in registers: RoPE, the
// subtraction of the channel mean and the first Hadamard level are four FMAs per channel pair
// (with p = cos + sin, m = cos - sin from the table: (x0 p + x1 m - (k0 + k1), x0 m - x1 p -
// (k0 - k1)) is the first butterfly of the rotated, centered pair); the remaining levels are
// register butterflies; one multiply by (top code / block maximum / sqrt(d)) and a saturating
// convert give the code.  The statistics and value items give a thread 8 channels of 16 (8 at
// d = 64) consecutive rows, so sums, maxima and the channel-major code rows need no transposition.
#include <cstdlib>

#include "vc_prep_common.cuh"

namespace vc {
namespace {

constexpr int kWorkers = 3;     // warpgroups per CTA
constexpr int kWT = 128;        // threads per worker = rows per item

enum : int { kKS = 0, kVS = 1, kQQ = 2, kKQ = 3, kVQ = 4 };

struct Fused {
  PrepArgs a;
  unsigned int *cnt;            // [BH] statistics items of the head that have finished
  unsigned int *ready;          // [BH] 1 once k_mean / v_scale / v_amax of the head are final
  unsigned int *abort_flag;     // set by the first wait that gives up
  unsigned int *status;
  int has_ks, stats_per_head, per_head, n_items;
  unsigned long long* prof;     // timing experiments only: [workers][8] cycles per phase (thread 0 of every worker)
  int dbg;                      // timing experiments only (wrong results): 1 = no loads, 2 = no item bodies
  int order;                    // 0: statistics, Q, quantization of one head after the other;
                                // 1: statistics one head ahead of the quantization
  unsigned int wait_limit;
};

struct Item {
  int kind, bh, blk;
};

// Position in the item sequence.  Items are numbered round by round.
//   order 0, round h:  [KS, VS of head h, blocks ascending] [QQ of head h] [KQ, VQ of head h, blocks descending]
//   order 1, round r:  [KS, VS of head r] [KQ, VQ of head r-1, ascending] [QQ of head r-1]   (r = 0 .. BH)
// A cursor moves forward by a fixed stride without divisions.
struct Cursor {
  int item, r, j;     // item number, round, index inside the round
};
__device__ __forceinline__ int round_len(const Fused& f, int r) {
  if (f.order == 0) return f.per_head;
  return (r < f.a.BH ? f.stats_per_head : 0) + (r >= 1 ? 3 * f.a.nb : 0);
}
__device__ __forceinline__ Cursor cursor_at(const Fused& f, int item) {
  Cursor c;
  c.item = item;
  if (f.order == 0 || item < f.stats_per_head) {
    c.r = f.order == 0 ? item / f.per_head : 0;
    c.j = item - c.r * f.per_head;
  } else {
    const int i2 = item - f.stats_per_head;
    c.r = 1 + i2 / f.per_head;
    c.j = i2 - (c.r - 1) * f.per_head;
  }
  return c;
}
__device__ __forceinline__ void advance(const Fused& f, Cursor& c, int stride) {
  c.item += stride;
  if (c.item >= f.n_items) return;
  c.j += stride;
  int len = round_len(f, c.r);
  while (c.j >= len) { c.j -= len; ++c.r; len = round_len(f, c.r); }
}
__device__ __forceinline__ Item item_of(const Fused& f, const Cursor& c) {
  Item it;
  const int nb = f.a.nb;
  int j = c.j;
  if (f.order == 0) {
    it.bh = c.r;
    if (j < f.stats_per_head) {
      if (f.has_ks) { it.blk = j >> 1; it.kind = (j & 1) ? kVS : kKS; }
      else { it.blk = j; it.kind = kVS; }
    } else if ((j -= f.stats_per_head) < nb) {
      it.blk = j; it.kind = kQQ;
    } else {
      j -= nb;
      it.blk = nb - 1 - (j >> 1);
      it.kind = (j & 1) ? kVQ : kKQ;
    }
  } else {
    const int ns = c.r < f.a.BH ? f.stats_per_head : 0;
    if (j < ns) {
      it.bh = c.r;
      if (f.has_ks) { it.blk = j >> 1; it.kind = (j & 1) ? kVS : kKS; }
      else { it.blk = j; it.kind = kVS; }
    } else if ((j -= ns) < 2 * nb) {
      it.bh = c.r - 1; it.blk = j >> 1; it.kind = (j & 1) ? kVQ : kKQ;
    } else {
      it.bh = c.r - 1; it.blk = j - 2 * nb; it.kind = kQQ;
    }
  }
  return it;
}

__device__ __forceinline__ void wbar(int wid) { asm volatile("bar.sync %0, %1;" ::"r"(wid + 1), "n"(kWT) : "memory"); }

__device__ __forceinline__ void cp_async16_zfill(void* dst, const void* src, int bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(dst)), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ unsigned int ld_acquire(const unsigned int* p) {
  unsigned int v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release(unsigned int* p, unsigned int v) {
  asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ unsigned int max_bf16x2(unsigned int a, unsigned int b) {
  unsigned int d;
  asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
__device__ __forceinline__ unsigned int min_bf16x2(unsigned int a, unsigned int b) {
  unsigned int d;
  asm("min.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
__device__ __forceinline__ unsigned long long gtime() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ float bf_lo(unsigned int w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(unsigned int w) { return __uint_as_float(w & 0xffff0000u); }

// Per-worker shared memory.
template <int D> struct WorkerSmem {
  static constexpr int kStage = kBlock * 2 * D;                 // one 128-row block of bf16
  static constexpr int kBytes = 2 * kStage + 2 * kBlock * 4 + 2 * D * 4 + 64;
  unsigned char* stage[2];
  int* psrc;        // [2][128] input row behind every row of the item in flight / the next one
  float* hk;        // [D] K: per pair -(k0 + k1), -(k0 - k1) (fused form) or the channel mean itself
  float* vinv;      // [D] V: 448 / amax per channel, 0 for a channel whose residual is zero
  float* red;       // [8] block maximum partials
  volatile int* flag;   // [2] "this worker folds the head's statistics", "the head's statistics are ready"
  __device__ WorkerSmem(unsigned char* base) {
    stage[0] = base; stage[1] = base + kStage;
    psrc = reinterpret_cast<int*>(base + 2 * kStage);
    hk = reinterpret_cast<float*>(psrc + 2 * kBlock);
    vinv = hk + D;
    red = vinv + D;
    flag = reinterpret_cast<volatile int*>(red + 8);
  }
};

template <int D> struct RopeSplit8;          // pair boundaries of the default channel split
template <> struct RopeSplit8<128> { static constexpr int p1 = 22, p2 = 43; };   // 44 / 42 / 42
template <> struct RopeSplit8<64> { static constexpr int p1 = 12, p2 = 22; };    // 24 / 20 / 20
template <int D> __device__ __forceinline__ constexpr int axis_of_pair(int p) {
  return p < RopeSplit8<D>::p1 ? 0 : (p < RopeSplit8<D>::p2 ? 1 : 2);
}

// Input row behind row `wt` of an item (-1: padding or no item).  K and V rows are gathered by pi
// in the passes that produce permuted output or per-block statistics of the permuted order; the
// entry is clamped into [0, N), so a bad permutation cannot become a bad address.
__device__ __forceinline__ int src_row_of(const Fused& f, const Cursor& c, int wt) {
  if (c.item >= f.n_items) return -1;
  const Item it = item_of(f, c);
  const int t = it.blk * kBlock + wt;
  if (t >= f.a.N) return -1;
  if (f.a.perm == nullptr || it.kind == kKS || it.kind == kQQ) return t;
  const int s = __ldg(&f.a.perm[(size_t)it.bh * f.a.N + t]);
  return min(max(s, 0), f.a.N - 1);
}

// Coalesced copy of an item's block into a stage: consecutive lanes take consecutive 16-byte
// chunks of a row; chunk c of row r lands at chunk position c ^ (r % 8) of the row (bank-conflict
// free for the row-per-thread reads as well as for the column-owner reads).
template <int D>
__device__ __forceinline__ void issue_loads(const Fused& f, const Cursor& c, unsigned char* stage, const int* psrc, int wt) {
  constexpr int CC = D / 8, RG = kWT / CC, RPT = kBlock / RG;
  static_assert(RG % 8 == 0, "row groups must keep r % 8 fixed per thread");
  if (c.item < f.n_items && !(f.dbg & 1)) {
    const PrepArgs& a = f.a;
    const Item it = item_of(f, c);
    const int b = it.bh / a.H, h = it.bh - b * a.H;
    const int col = wt % CC, rg = wt / CC;
    const __nv_bfloat16* base = (it.kind == kQQ ? a.q : (it.kind == kKS || it.kind == kKQ) ? a.k : a.v) +
                                b * a.stride_b + h * a.stride_h + 8 * col;
    unsigned char* dst = stage + rg * (2 * D) + ((col ^ (rg & 7)) << 4);
#pragma unroll
    for (int k = 0; k < RPT; ++k) {
      const int sr = psrc[rg + RG * k];
      cp_async16_zfill(dst + k * (RG * 2 * D), base + (int64_t)(sr < 0 ? 0 : sr) * a.stride_n, sr < 0 ? 0 : 16);
    }
  }
  cp_async_commit();
}

// Bounded wait for a head's statistics (one thread of the worker).
__device__ __forceinline__ bool wait_ready(const Fused& f, int bh) {
  if (f.prof) atomicMin(&f.prof[444 * 8 + (size_t)bh * 4 + 2], gtime());     // first consumer arrives
  if (ld_acquire(&f.ready[bh])) return true;
  for (unsigned int i = 0; i < f.wait_limit; ++i) {
    __nanosleep(i < 64 ? 100 : 400);
    if (ld_acquire(&f.ready[bh])) return true;
    if ((i & 15u) == 15u && *reinterpret_cast<volatile unsigned int*>(f.abort_flag)) return false;
  }
  atomicExch(f.abort_flag, 1u);
  atomicExch(f.status, kStatusTimeout | 0x50u);
  return false;
}

// ---------------------------------------------------------------------------------------
// After a statistics item: count it; the worker that finishes a head's last one folds the
// partial results (fixed order, so the result does not depend on which worker that is).
template <int D>
__device__ __forceinline__ void stats_done(const Fused& f, WorkerSmem<D>& ws, unsigned char* scratch, int bh, int wt, int wid) {
  const PrepArgs& a = f.a;
  __threadfence();
  wbar(wid);
  if (wt == 0) *ws.flag = atomicAdd(&f.cnt[bh], 1u) == (unsigned int)(f.stats_per_head - 1);
  wbar(wid);
  if (!*ws.flag) return;
  if (f.prof && wt == 0) f.prof[444 * 8 + (size_t)bh * 4 + 0] = gtime();
  __threadfence();
  // channel sums of the head: nb partial rows of D floats.  A thread takes four channels of
  // every SL-th row (many independent loads in flight), the SL slices meet in fixed order.
  constexpr int CQ = D / 4, SL = kWT / CQ;
  double* slice = reinterpret_cast<double*>(scratch);            // [SL][D]
  if (f.has_ks) {
    const int cq = wt % CQ, sl = wt / CQ;
    const float4* kp = reinterpret_cast<const float4*>(a.k_part + (size_t)bh * a.nb * D) + cq;
    double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
    int j = sl;
    for (; j + 7 * SL < a.nb; j += 8 * SL) {
      float4 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) v[u] = __ldcg(kp + (size_t)(j + u * SL) * CQ);
#pragma unroll
      for (int u = 0; u < 8; ++u) { s0 += (double)v[u].x; s1 += (double)v[u].y; s2 += (double)v[u].z; s3 += (double)v[u].w; }
    }
    for (; j < a.nb; j += SL) {
      const float4 v = __ldcg(kp + (size_t)j * CQ);
      s0 += (double)v.x; s1 += (double)v.y; s2 += (double)v.z; s3 += (double)v.w;
    }
    double* dst = slice + sl * D + 4 * cq;
    dst[0] = s0; dst[1] = s1; dst[2] = s2; dst[3] = s3;
  }
  wbar(wid);
  if (wt < D) {
    double s = 0.0;
    if (f.has_ks) {
#pragma unroll
      for (int g = 0; g < SL; ++g) s += slice[g * D + wt];
    }
    a.k_mean[(size_t)bh * D + wt] = (float)(s / (double)a.N);
    const float am = __uint_as_float(__ldcg(&a.v_amax[(size_t)bh * D + wt]));
    a.v_scale[(size_t)bh * D + wt] = am > 0.f ? am / 448.0f : 1.0f;
  }
  __threadfence();
  wbar(wid);
  if (wt == 0) st_release(&f.ready[bh], 1u);
  if (f.prof && wt == 0) f.prof[444 * 8 + (size_t)bh * 4 + 1] = gtime();
}

// ---------------------------------------------------------------------------------------
// KS: column sums of RoPE(K) over the block's rows (the channel mean is taken after the rotation
// and needs no gather: it is a sum over all rows).
template <int D, bool FAST>
__device__ __forceinline__ void ks_item(const Fused& f, WorkerSmem<D>& ws, const float2* tab, const Item& it,
                                        unsigned char* stage, int wt, int wid) {
  constexpr int CC = D / 8, RG = kWT / CC, RPT = kBlock / RG;
  const PrepArgs& a = f.a;
  const int col = wt % CC, rg = wt / CC, row0 = rg * RPT;
  const int n_valid = min(kBlock, a.N - it.blk * kBlock);
  const bool do_rope = a.flags & VC_FLAG_ROPE;
  // table cursor of each of the thread's four channel pairs and its steps: along x, when x wraps,
  // when x and y wrap
  int idx[4], dx[4], dwx[4], dwy[4];
  int tt = 0, ty = 0, tx = 0;
  if (do_rope) {
    grid_pos(a.rd, min(it.blk * kBlock + row0, a.N - 1), tt, ty, tx);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int p = 4 * col + j;
      const int ax = p >= a.rd.pair_start[2] ? 2 : (p >= a.rd.pair_start[1] ? 1 : 0);
      const int pairs = a.rd.pairs[ax];
      idx[j] = a.rd.off[ax] + (p - a.rd.pair_start[ax]) + (ax == 0 ? tt : ax == 1 ? ty : tx) * pairs;
      dx[j] = ax == 2 ? pairs : 0;
      dwx[j] = ax == 2 ? -(a.rd.grid_w - 1) * pairs : (ax == 1 ? pairs : 0);
      dwy[j] = ax == 2 ? -(a.rd.grid_w - 1) * pairs : (ax == 1 ? -(a.rd.grid_h - 1) * pairs : pairs);
    }
  }
  float acc[16];
#pragma unroll
  for (int c = 0; c < 16; ++c) acc[c] = 0.f;
#pragma unroll 4
  for (int i = 0; i < RPT; ++i) {
    const int r = row0 + i;
    if (r >= n_valid) break;
    const uint4 raw = *reinterpret_cast<const uint4*>(stage + r * (2 * D) + ((col ^ (r & 7)) << 4));
    const unsigned int w[4] = {raw.x, raw.y, raw.z, raw.w};
    if (do_rope) {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float2 e = tab[idx[j]];
        const float x0 = bf_lo(w[j]), x1 = bf_hi(w[j]);
        if (FAST) {       // e = (cos + sin, cos - sin): four plain sums, combined below
          acc[4 * j] = fmaf(x0, e.x, acc[4 * j]);
          acc[4 * j + 1] = fmaf(x0, e.y, acc[4 * j + 1]);
          acc[4 * j + 2] = fmaf(x1, e.x, acc[4 * j + 2]);
          acc[4 * j + 3] = fmaf(x1, e.y, acc[4 * j + 3]);
        } else {          // e = (cos, sin)
          acc[4 * j] = fmaf(x0, e.x, acc[4 * j]);
          acc[4 * j + 1] = fmaf(x1, e.y, acc[4 * j + 1]);
          acc[4 * j + 2] = fmaf(x0, e.y, acc[4 * j + 2]);
          acc[4 * j + 3] = fmaf(x1, e.x, acc[4 * j + 3]);
        }
      }
      if (++tx == a.rd.grid_w) {
        tx = 0;
        if (++ty == a.rd.grid_h) {
          ty = 0;
#pragma unroll
          for (int j = 0; j < 4; ++j) idx[j] += dwy[j];
        } else {
#pragma unroll
          for (int j = 0; j < 4; ++j) idx[j] += dwx[j];
        }
      } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) idx[j] += dx[j];
      }
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j) { acc[4 * j] += bf_lo(w[j]); acc[4 * j + 2] += bf_hi(w[j]); }
    }
  }
  float s[8];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    if (!do_rope) { s[2 * j] = acc[4 * j]; s[2 * j + 1] = acc[4 * j + 2]; }
    else if (FAST) {
      // sum(x0 c - x1 s) and sum(x0 s + x1 c) from the sums against p = c + s and m = c - s
      s[2 * j] = 0.5f * ((acc[4 * j] + acc[4 * j + 1]) - (acc[4 * j + 2] - acc[4 * j + 3]));
      s[2 * j + 1] = 0.5f * ((acc[4 * j] - acc[4 * j + 1]) + (acc[4 * j + 2] + acc[4 * j + 3]));
    } else {
      s[2 * j] = acc[4 * j] - acc[4 * j + 1];
      s[2 * j + 1] = acc[4 * j + 2] + acc[4 * j + 3];
    }
  }
  wbar(wid);                                  // every thread is done reading the stage
  float* part = reinterpret_cast<float*>(stage);     // [RG][D]
  *reinterpret_cast<float4*>(part + rg * D + 8 * col) = make_float4(s[0], s[1], s[2], s[3]);
  *reinterpret_cast<float4*>(part + rg * D + 8 * col + 4) = make_float4(s[4], s[5], s[6], s[7]);
  wbar(wid);
  if (wt < D) {
    float t = 0.f;
#pragma unroll
    for (int g = 0; g < RG; ++g) t += part[g * D + wt];
    a.k_part[((size_t)it.bh * a.nb + it.blk) * D + wt] = t;
  }
  stats_done<D>(f, ws, stage, it.bh, wt, wid);
}

// ---------------------------------------------------------------------------------------
// VS: block mean (Eq. 4) and the block's contribution to the per-channel maximum of the residual.
// max |v - mu| over the block = max(max v - mu, mu - min v), and rounding is monotone, so the
// maximum and minimum of the bf16 values (exact, two per instruction) are all that is needed.
template <int D>
__device__ __forceinline__ void vs_item(const Fused& f, WorkerSmem<D>& ws, const Item& it, unsigned char* stage, int wt, int wid) {
  constexpr int CC = D / 8, RG = kWT / CC, RPT = kBlock / RG;
  const PrepArgs& a = f.a;
  const int col = wt % CC, rg = wt / CC, row0 = rg * RPT;
  const int n_valid = min(kBlock, a.N - it.blk * kBlock);
  float s[8];
  unsigned int mx[4], mn[4];
#pragma unroll
  for (int c = 0; c < 8; ++c) s[c] = 0.f;
#pragma unroll
  for (int j = 0; j < 4; ++j) { mx[j] = 0xff80ff80u; mn[j] = 0x7f807f80u; }     // -inf, +inf
#pragma unroll 4
  for (int i = 0; i < RPT; ++i) {
    const int r = row0 + i;
    if (r >= n_valid) break;
    const uint4 raw = *reinterpret_cast<const uint4*>(stage + r * (2 * D) + ((col ^ (r & 7)) << 4));
    const unsigned int w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      s[2 * j] += bf_lo(w[j]);
      s[2 * j + 1] += bf_hi(w[j]);
      mx[j] = max_bf16x2(mx[j], w[j]);
      mn[j] = min_bf16x2(mn[j], w[j]);
    }
  }
  wbar(wid);                                  // every thread is done reading the stage
  float* psum = reinterpret_cast<float*>(stage);                               // [RG][D]
  unsigned int* pmx = reinterpret_cast<unsigned int*>(stage + RG * D * 4);     // [RG][D / 2]
  unsigned int* pmn = pmx + RG * (D / 2);
  *reinterpret_cast<float4*>(psum + rg * D + 8 * col) = make_float4(s[0], s[1], s[2], s[3]);
  *reinterpret_cast<float4*>(psum + rg * D + 8 * col + 4) = make_float4(s[4], s[5], s[6], s[7]);
  *reinterpret_cast<uint4*>(pmx + rg * (D / 2) + 4 * col) = make_uint4(mx[0], mx[1], mx[2], mx[3]);
  *reinterpret_cast<uint4*>(pmn + rg * (D / 2) + 4 * col) = make_uint4(mn[0], mn[1], mn[2], mn[3]);
  wbar(wid);
  if (wt < D) {
    float t = 0.f, hi = -INFINITY, lo = INFINITY;
#pragma unroll
    for (int g = 0; g < RG; ++g) {
      t += psum[g * D + wt];
      const unsigned int wx = pmx[g * (D / 2) + (wt >> 1)], wn = pmn[g * (D / 2) + (wt >> 1)];
      hi = fmaxf(hi, (wt & 1) ? bf_hi(wx) : bf_lo(wx));
      lo = fminf(lo, (wt & 1) ? bf_hi(wn) : bf_lo(wn));
    }
    const float mu = (a.flags & VC_FLAG_V_SMOOTH) ? t / (float)n_valid : 0.f;
    const float am = fmaxf(hi - mu, mu - lo);
    a.v_mu[((size_t)it.bh * a.nb + it.blk) * D + wt] = mu;
    atomicMax(&a.v_amax[(size_t)it.bh * D + wt], __float_as_uint(fmaxf(am, 0.f)));
  }
  stats_done<D>(f, ws, stage, it.bh, wt, wid);
}

// ---------------------------------------------------------------------------------------
// VQ: residual against the block mean, per-channel scale, E4M3 codes written channel-major
// (token-contiguous), block means stored divided by the scale (App. B).
template <int D>
__device__ __forceinline__ void vq_item(const Fused& f, WorkerSmem<D>& ws, const Item& it, unsigned char* stage, int wt, int wid) {
  constexpr int CC = D / 8, RG = kWT / CC, RPT = kBlock / RG, WPC = RPT / 4;    // code words per channel and thread
  const PrepArgs& a = f.a;
  const int col = wt % CC, rg = wt / CC, row0 = rg * RPT;
  const int n_valid = min(kBlock, a.N - it.blk * kBlock);
  const size_t mu_at = ((size_t)it.bh * a.nb + it.blk) * D + 8 * col;
  float mu[8], inv[8];
  {
    const float4 m0 = __ldcg(reinterpret_cast<const float4*>(a.v_mu + mu_at)), m1 = __ldcg(reinterpret_cast<const float4*>(a.v_mu + mu_at + 4));
    mu[0] = m0.x; mu[1] = m0.y; mu[2] = m0.z; mu[3] = m0.w; mu[4] = m1.x; mu[5] = m1.y; mu[6] = m1.z; mu[7] = m1.w;
    const float4 i0 = *reinterpret_cast<const float4*>(ws.vinv + 8 * col), i1 = *reinterpret_cast<const float4*>(ws.vinv + 8 * col + 4);
    inv[0] = i0.x; inv[1] = i0.y; inv[2] = i0.z; inv[3] = i0.w; inv[4] = i1.x; inv[5] = i1.y; inv[6] = i1.z; inv[7] = i1.w;
  }
  unsigned int cw[8][WPC];
#pragma unroll
  for (int k = 0; k < 8; ++k)
#pragma unroll
    for (int q = 0; q < WPC; ++q) cw[k][q] = 0u;
#pragma unroll
  for (int i = 0; i < RPT; i += 2) {
    const int r0 = row0 + i, r1 = r0 + 1;
    const uint4 ra = *reinterpret_cast<const uint4*>(stage + r0 * (2 * D) + ((col ^ (r0 & 7)) << 4));
    const uint4 rb = *reinterpret_cast<const uint4*>(stage + r1 * (2 * D) + ((col ^ (r1 & 7)) << 4));
    const unsigned int wa[4] = {ra.x, ra.y, ra.z, ra.w}, wb[4] = {rb.x, rb.y, rb.z, rb.w};
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const float va = (k & 1) ? bf_hi(wa[k >> 1]) : bf_lo(wa[k >> 1]);
      const float vb = (k & 1) ? bf_hi(wb[k >> 1]) : bf_lo(wb[k >> 1]);
      // R = V' - mu (Eq. 4), then one multiply by 448 / amax and the saturating convert
      const unsigned int two = __nv_cvt_float2_to_fp8x2(make_float2((va - mu[k]) * inv[k], (vb - mu[k]) * inv[k]), __NV_SATFINITE, __NV_E4M3);
      cw[k][i >> 2] |= two << (8 * (i & 2));
    }
  }
  if (n_valid < kBlock) {                     // padding rows of the ragged last block: code 0
#pragma unroll
    for (int q = 0; q < WPC; ++q) {
      const int left = n_valid - (row0 + 4 * q);      // valid tokens among this word's four
      const unsigned int mask = left >= 4 ? 0xffffffffu : (left <= 0 ? 0u : (1u << (8 * left)) - 1u);
#pragma unroll
      for (int k = 0; k < 8; ++k) cw[k][q] &= mask;
    }
  }
  if (rg == 0) {                              // block means, divided by the value scale
    unsigned int mw[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float m0 = mu[2 * j] * (inv[2 * j] > 0.f ? inv[2 * j] : 1.0f), m1 = mu[2 * j + 1] * (inv[2 * j + 1] > 0.f ? inv[2 * j + 1] : 1.0f);
      const __nv_bfloat162 h2 = __floats2bfloat162_rn(m0, m1);
      mw[j] = *reinterpret_cast<const unsigned int*>(&h2);
    }
    *reinterpret_cast<uint4*>(a.v_means + mu_at) = make_uint4(mw[0], mw[1], mw[2], mw[3]);
  }
  wbar(wid);                                  // every thread is done reading the stage
  // code tile [D channels][128 tokens]; 16-byte chunk c of channel ch at position c ^ ((ch / 8) % 8)
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const int ch = 8 * col + k;
    if constexpr (WPC == 4) {
      *reinterpret_cast<uint4*>(stage + ch * kBlock + ((rg ^ (col & 7)) << 4)) = make_uint4(cw[k][0], cw[k][1], cw[k][2], cw[k][3]);
    } else {
      static_assert(WPC == 2, "tokens per thread");
      *reinterpret_cast<uint2*>(stage + ch * kBlock + (((rg >> 1) ^ (col & 7)) << 4) + 8 * (rg & 1)) = make_uint2(cw[k][0], cw[k][1]);
    }
  }
  wbar(wid);
  uint8_t* gdst = a.v_codes + (size_t)it.bh * D * a.n_pad + (size_t)it.blk * kBlock;
#pragma unroll
  for (int c = 0; c < D * 8 / kWT; ++c) {
    const int idx = c * kWT + wt, ch = idx >> 3, chunk = idx & 7;
    const uint4 v = *reinterpret_cast<const uint4*>(stage + ch * kBlock + ((chunk ^ ((ch >> 3) & 7)) << 4));
    *reinterpret_cast<uint4*>(gdst + (size_t)ch * a.n_pad + 16 * chunk) = v;
  }
}

// ---------------------------------------------------------------------------------------
// QQ / KQ: one row per thread.
template <int D, bool FAST, bool INT8>
__device__ __forceinline__ void row_item(const Fused& f, WorkerSmem<D>& ws, const float2* tab, const float* zeros, const Item& it,
                                         unsigned char* stage, int src_row, int iter, int wt, int wid) {
  const PrepArgs& a = f.a;
  const bool isK = it.kind == kKQ;
  const int row = wt, lane = wt & 31, warp = wt >> 5;
  const bool valid = src_row >= 0;
  const bool center = isK && f.has_ks;
  float x[D];
#pragma unroll
  for (int i = 0; i < D / 8; ++i) {
    const uint4 raw = *reinterpret_cast<const uint4*>(stage + row * (2 * D) + ((i ^ (row & 7)) << 4));
    const unsigned int w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) { x[8 * i + 2 * j] = bf_lo(w[j]); x[8 * i + 2 * j + 1] = bf_hi(w[j]); }
  }
  int tt, ty, tx;
  grid_pos(a.rd, valid ? src_row : 0, tt, ty, tx);
  // entry of pair p of axis ax: off[ax] + pos[ax] * pairs[ax] + (p - pair_start[ax])
  const int e0 = a.rd.off[0] + tt * a.rd.pairs[0] - a.rd.pair_start[0], e1 = a.rd.off[1] + ty * a.rd.pairs[1] - a.rd.pair_start[1],
            e2 = a.rd.off[2] + tx * a.rd.pairs[2] - a.rd.pair_start[2];
  if constexpr (FAST) {
    // RoPE, mean subtraction and the first Hadamard level in four FMAs per pair
    const float4* nk = reinterpret_cast<const float4*>(center ? ws.hk : zeros);
#pragma unroll
    for (int i = 0; i < D / 2; i += 2) {
      const float4 k4 = nk[i >> 1];
      const float2 pm0 = tab[(axis_of_pair<D>(i) == 0 ? e0 : axis_of_pair<D>(i) == 1 ? e1 : e2) + i];
      const float2 pm1 = tab[(axis_of_pair<D>(i + 1) == 0 ? e0 : axis_of_pair<D>(i + 1) == 1 ? e1 : e2) + i + 1];
      float x0 = x[2 * i], x1 = x[2 * i + 1];
      x[2 * i] = fmaf(x1, pm0.y, fmaf(x0, pm0.x, k4.x));
      x[2 * i + 1] = fmaf(-x1, pm0.x, fmaf(x0, pm0.y, k4.y));
      x0 = x[2 * i + 2]; x1 = x[2 * i + 3];
      x[2 * i + 2] = fmaf(x1, pm1.y, fmaf(x0, pm1.x, k4.z));
      x[2 * i + 3] = fmaf(-x1, pm1.x, fmaf(x0, pm1.y, k4.w));
    }
    if (!valid) {
#pragma unroll
      for (int c = 0; c < D; ++c) x[c] = 0.f;
    }
#pragma unroll
    for (int sft = 2; sft < D; sft <<= 1) {
#pragma unroll
      for (int c = 0; c < D; ++c) {
        if (!(c & sft)) {
          const float u = x[c], v = x[c | sft];
          x[c] = u + v;
          x[c | sft] = u - v;
        }
      }
    }
  } else {
    if ((a.flags & VC_FLAG_ROPE) && valid) {
#pragma unroll
      for (int i = 0; i < D / 2; ++i) {
        const int eb = i < a.rd.pair_start[1] ? e0 : (i < a.rd.pair_start[2] ? e1 : e2);
        const float2 cs = a.rope_in_smem ? tab[eb + i] : __ldg(&a.rope[eb + i]);
        const float x0 = x[2 * i], x1 = x[2 * i + 1];
        x[2 * i] = x0 * cs.x - x1 * cs.y;
        x[2 * i + 1] = x0 * cs.y + x1 * cs.x;
      }
    }
    if (center && valid) {
      const float4* km = reinterpret_cast<const float4*>(ws.hk);
#pragma unroll
      for (int c4 = 0; c4 < D / 4; ++c4) {
        const float4 m = km[c4];
        x[4 * c4] -= m.x; x[4 * c4 + 1] -= m.y; x[4 * c4 + 2] -= m.z; x[4 * c4 + 3] -= m.w;
      }
    }
    if (a.flags & VC_FLAG_HADAMARD) {
#pragma unroll
      for (int sft = 1; sft < D; sft <<= 1) {
#pragma unroll
        for (int c = 0; c < D; ++c) {
          if (!(c & sft)) {
            const float u = x[c], v = x[c | sft];
            x[c] = u + v;
            x[c | sft] = u - v;
          }
        }
      }
    }
  }
  const float rs = (FAST || (a.flags & VC_FLAG_HADAMARD)) ? (D == 128 ? 0.08838834764831845f : 0.125f) : 1.0f;   // 1 / sqrt(D)
  float m0 = 0.f, m1 = 0.f;
#pragma unroll
  for (int c = 0; c < D; c += 4) {
    m0 = max3(m0, fabsf(x[c]), fabsf(x[c + 1]));
    m1 = max3(m1, fabsf(x[c + 2]), fabsf(x[c + 3]));
  }
  float amax = warp_max(fmaxf(m0, m1) * rs);   // the maximum and the (positive) scale commute exactly
  float* rbuf = ws.red + 4 * (iter & 1);
  if (lane == 0) rbuf[warp] = amax;
  wbar(wid);                                   // also: every thread has its row in registers
  amax = fmaxf(fmaxf(rbuf[0], rbuf[1]), fmaxf(rbuf[2], rbuf[3]));
  const float top = INT8 ? 127.0f : 448.0f;
  const float inv = amax > 0.f ? top / amax : 0.f;
  if (wt == 0) (isK ? a.k_scale : a.q_scale)[(size_t)it.bh * a.nb + it.blk] = amax > 0.f ? amax / top : 1.0f;
  const float sc = rs * inv;
  // codes into the (now free) stage as a swizzled tile; the worker copies it out with coalesced stores
  constexpr int CPR = D / 16;
  uint4* dst = reinterpret_cast<uint4*>(stage + row * D);
  const int sw = (row / (8 / CPR)) & (CPR - 1);
#pragma unroll
  for (int i = 0; i < D / 16; ++i) {
    unsigned int w[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int c = 16 * i + 4 * j;
      if constexpr (INT8) {
        // |y| <= 127: adding 1.5 * 2^23 rounds y to the nearest even integer in the low mantissa
        // bits, two's complement for negative values; the low bytes are the codes
        const unsigned int r0 = __float_as_uint(fmaf(x[c], sc, 12582912.0f)), r1 = __float_as_uint(fmaf(x[c + 1], sc, 12582912.0f));
        const unsigned int r2 = __float_as_uint(fmaf(x[c + 2], sc, 12582912.0f)), r3 = __float_as_uint(fmaf(x[c + 3], sc, 12582912.0f));
        w[j] = __byte_perm(__byte_perm(r0, r1, 0x0040), __byte_perm(r2, r3, 0x0040), 0x5410);
      } else {
        const unsigned int lo = __nv_cvt_float2_to_fp8x2(make_float2(x[c] * sc, x[c + 1] * sc), __NV_SATFINITE, __NV_E4M3);
        const unsigned int hi = __nv_cvt_float2_to_fp8x2(make_float2(x[c + 2] * sc, x[c + 3] * sc), __NV_SATFINITE, __NV_E4M3);
        w[j] = lo | (hi << 16);
      }
    }
    dst[i ^ sw] = make_uint4(w[0], w[1], w[2], w[3]);
  }
  wbar(wid);                                   // the code tile is complete
  uint8_t* gdst = (isK ? a.k_codes : a.q_codes) + ((size_t)it.bh * a.n_pad + (size_t)it.blk * kBlock) * D;
#pragma unroll
  for (int c = 0; c < CPR; ++c) {
    const int idx = c * kWT + wt, r = idx / CPR, chunk = idx % CPR;
    const int s2 = (r / (8 / CPR)) & (CPR - 1);
    const uint4 v = *reinterpret_cast<const uint4*>(stage + r * D + ((chunk ^ s2) << 4));
    *reinterpret_cast<uint4*>(gdst + (size_t)idx * 16) = v;
  }
}

// ---------------------------------------------------------------------------------------
template <int D, bool FAST, bool INT8>
__global__ void __launch_bounds__(kWorkers * kWT, 1) prep8_kernel(const Fused f) {
  extern __shared__ __align__(1024) unsigned char smem[];
  const PrepArgs& a = f.a;
  const int wid = threadIdx.x / kWT, wt = threadIdx.x % kWT;
  WorkerSmem<D> ws(smem + wid * WorkerSmem<D>::kBytes);
  float* zeros = reinterpret_cast<float*>(smem + kWorkers * WorkerSmem<D>::kBytes);   // [D]
  float2* tab_s = reinterpret_cast<float2*>(zeros + D);
  const float2* tab = a.rope;
  if ((a.flags & VC_FLAG_ROPE) && a.rope_in_smem) {
    for (int e = threadIdx.x; e < a.rd.entries; e += blockDim.x) {
      const float2 cs = __ldg(&a.rope[e]);
      tab_s[e] = FAST ? make_float2(cs.x + cs.y, cs.x - cs.y) : cs;
    }
    tab = tab_s;
  }
  if (threadIdx.x < D) zeros[threadIdx.x] = 0.f;
  __syncthreads();

  const int stride = gridDim.x * kWorkers;
  Cursor cur = cursor_at(f, blockIdx.x * kWorkers + wid);        // the item at hand
  Cursor nxt = cur, far = cur;                                   // the next one; the one three ahead
  advance(f, nxt, stride);
  far = nxt;
  advance(f, far, stride);
  ws.psrc[wt] = src_row_of(f, cur, wt);
  ws.psrc[kBlock + wt] = src_row_of(f, nxt, wt);
  int pre = src_row_of(f, far, wt);
  advance(f, far, stride);
  wbar(wid);
  issue_loads<D>(f, cur, ws.stage[0], ws.psrc, wt);
  int head_k = -1, head_v = -1, head_ready = -1;
  unsigned long long tacc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  long long t0 = clock64();
  auto lap = [&](int slot) { if (f.prof && wt == 0) { const long long t1 = clock64(); tacc[slot] += (unsigned long long)(t1 - t0); t0 = t1; } };
  for (int i = 0; cur.item < f.n_items; ++i) {
    const Item it = item_of(f, cur);
    const bool needs = (it.kind == kKQ && f.has_ks) || it.kind == kVQ;
    lap(0);
    if (needs && head_ready != it.bh && wt == 0) ws.flag[1] = wait_ready(f, it.bh) ? 1 : 0;
    lap(1);
    cp_async_wait<0>();                        // my chunks of this item have landed ...
    wbar(wid);                                 // ... and everyone's; the previous item is finished
    lap(2);
    if (needs && head_ready != it.bh) {
      if (!ws.flag[1]) break;                  // a wait gave up (status word written): stop this worker
      head_ready = it.bh;
    }
    issue_loads<D>(f, nxt, ws.stage[(i + 1) & 1], ws.psrc + ((i + 1) & 1) * kBlock, wt);
    unsigned char* stage = ws.stage[i & 1];
    const int my_src = ws.psrc[(i & 1) * kBlock + wt];
    if (it.kind == kKQ && f.has_ks && head_k != it.bh) {
      // the head's channel mean, in the form the row body adds it
      if (wt < D / 2) {
        const float2 km = __ldcg(reinterpret_cast<const float2*>(a.k_mean + (size_t)it.bh * D) + wt);
        *reinterpret_cast<float2*>(ws.hk + 2 * wt) = FAST ? make_float2(-(km.x + km.y), -(km.x - km.y)) : km;
      }
      head_k = it.bh;
      wbar(wid);
    }
    if (it.kind == kVQ && head_v != it.bh) {
      if (wt < D) {
        const float am = __uint_as_float(__ldcg(&a.v_amax[(size_t)it.bh * D + wt]));
        ws.vinv[wt] = am > 0.f ? 448.0f / am : 0.f;
      }
      head_v = it.bh;
      wbar(wid);
    }
    lap(3);
    if (f.dbg & 2) { if (it.kind == kKS || it.kind == kVS) stats_done<D>(f, ws, stage, it.bh, wt, wid); }
    else if (it.kind == kKS) ks_item<D, FAST>(f, ws, tab, it, stage, wt, wid);
    else if (it.kind == kVS) vs_item<D>(f, ws, it, stage, wt, wid);
    else if (it.kind == kVQ) vq_item<D>(f, ws, it, stage, wt, wid);
    else row_item<D, FAST, INT8>(f, ws, tab, zeros, it, stage, my_src, i, wt, wid);
    lap(it.kind == kKS || it.kind == kVS ? 4 : (it.kind == kVQ ? 5 : 6));
    ws.psrc[(i & 1) * kBlock + wt] = pre;      // rows of the item after the next
    pre = src_row_of(f, far, wt);
    cur = nxt;
    advance(f, nxt, stride);
    advance(f, far, stride);
    lap(7);
  }
  if (f.prof && wt == 0)
    for (int q = 0; q < 8; ++q) f.prof[(size_t)(blockIdx.x * kWorkers + wid) * 8 + q] = tacc[q];
  cp_async_wait<0>();                          // nothing of mine is in flight when the CTA exits
}

// Validator of the permutation (VC_FLAG_CHECK_PERM): every entry inside [0, N) and none twice.
__global__ void perm_check_kernel(const int32_t* __restrict__ perm, unsigned int* bits, unsigned int* status, int N,
                                  int words_per_head, size_t total) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  const int bh = (int)(i / (size_t)N);
  const int v = perm[i];
  if (v < 0 || v >= N) { atomicOr(status, kStatusBadPerm | 1u); return; }
  const unsigned int bit = 1u << (v & 31);
  if (atomicOr(&bits[(size_t)bh * words_per_head + (v >> 5)], bit) & bit) atomicOr(status, kStatusBadPerm | 2u);
}

int prep8_order() {
  static int order = -1;
  if (order < 0) {
    const char* e = getenv("VC_PREP_ORDER");
    order = e ? atoi(e) : 0;
  }
  return order;
}

int sm_count() {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
    sms = 148;
  return sms;
}

template <int D, bool FAST, bool INT8>
cudaError_t launch(const Fused& f, size_t smem, cudaStream_t s) {
  cudaError_t e = cudaFuncSetAttribute(prep8_kernel<D, FAST, INT8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int ctas = (f.n_items + kWorkers - 1) / kWorkers;
  const int sms = sm_count();
  prep8_kernel<D, FAST, INT8><<<ctas < sms ? ctas : sms, kWorkers * kWT, smem, s>>>(f);
  return cudaGetLastError();
}

template <int D>
cudaError_t run8(const Problem& pr, Fused f, cudaStream_t s) {
  const PrepArgs& a = f.a;
  const bool all_on = (a.flags & (VC_FLAG_ROPE | VC_FLAG_HADAMARD)) == (VC_FLAG_ROPE | VC_FLAG_HADAMARD);   // the fused row body
  const size_t base = (size_t)kWorkers * WorkerSmem<D>::kBytes + D * 4;
  const size_t rope_bytes = (a.flags & VC_FLAG_ROPE) ? (size_t)a.rd.entries * 8 : 0;
  const bool fits = base + rope_bytes <= 227 * 1024;
  f.a.rope_in_smem = fits;
  const bool fast = all_on && a.rope_default && fits;
  const size_t smem = base + (fits ? rope_bytes : 0);
  const bool int8 = a.flags & VC_FLAG_INT8_QK;
  if (fast) return int8 ? launch<D, true, true>(f, smem, s) : launch<D, true, false>(f, smem, s);
  return int8 ? launch<D, false, true>(f, smem, s) : launch<D, false, false>(f, smem, s);
}

}  // namespace

cudaError_t launch_perm_check(const Problem& pr, const int32_t* perm, const WorkLayout& wl, uint8_t* work, cudaStream_t s) {
  if (!(pr.flags & VC_FLAG_CHECK_PERM) || !perm) return cudaSuccess;
  cudaError_t e = cudaMemsetAsync(work + wl.perm_bits, 0, wl.perm_bits_bytes, s);
  if (e != cudaSuccess) return e;
  const size_t total = (size_t)pr.BH * pr.N;
  perm_check_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(perm, reinterpret_cast<unsigned int*>(work + wl.perm_bits),
                                                                    reinterpret_cast<unsigned int*>(work + wl.status), pr.N,
                                                                    (pr.N + 31) / 32, total);
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t launch_prep8(const Problem& pr, const PrepArgs& a, const WorkLayout& wl, uint8_t* work, cudaStream_t s) {
  Fused f{};
  f.a = a;
  unsigned int* sync = reinterpret_cast<unsigned int*>(work + wl.sync);
  f.cnt = sync;
  f.ready = sync + pr.BH;
  f.abort_flag = sync + 2 * (size_t)pr.BH;
  f.status = reinterpret_cast<unsigned int*>(work + wl.status);
  f.has_ks = (pr.flags & VC_FLAG_K_SMOOTH) ? 1 : 0;
  f.stats_per_head = (f.has_ks ? 2 : 1) * pr.nb;
  f.per_head = f.stats_per_head + 3 * pr.nb;
  if ((int64_t)f.per_head * pr.BH > 0x7ff00000LL) return cudaErrorInvalidValue;
  f.n_items = f.per_head * pr.BH;
  f.order = prep8_order();
  { const char* e = getenv("VC_PREP_DBG"); f.dbg = e ? atoi(e) : 0; }
  { const char* e = getenv("VC_PREP_PROF"); f.prof = e ? reinterpret_cast<unsigned long long*>(strtoull(e, nullptr, 0)) : nullptr; }
  const uint32_t lim = wait_limit_override();
  f.wait_limit = lim ? lim : (1u << 21);               // x 0.4 us: about a second
  cudaError_t e;
  if ((e = cudaMemsetAsync(work + wl.sync, 0, wl.sync_bytes, s)) != cudaSuccess) return e;
  e = pr.d == 128 ? run8<128>(pr, f, s) : run8<64>(pr, f, s);
  count_launches(1);
  return e;
}

}  // namespace vc
