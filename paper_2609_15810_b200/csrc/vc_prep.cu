// Fused preprocessing pass of VC-Attention for sm_100a (Sec. 3.4 "Fused preprocessing",
// App. B): every operand is read as bf16 with 16-byte vector loads and leaves as low-bit
// codes plus scales; no rotated / permuted / centered high-precision tensor reaches HBM.
//
//   Q : RoPE -> Hadamard (in registers, a row in two threads) -> per-128-row scale -> codes
//   K : RoPE -> column sums (stats launch) ... gather by pi -> RoPE at the source position
//       -> subtract channel mean -> Hadamard -> scale -> codes
//   V : gather by pi -> block mean (Eq. 4) and residual amax (stats launch) ...
//       gather -> residual -> codes written channel-major, block means beside them
//
// The two global reductions (K channel mean over all tokens, per-channel amax of the V
// residual over all tokens) force statistics launches before the quantizing launches; heads
// can be processed in groups so that the second read of K and V may hit L2.  All passes are
// persistent kernels that prefetch the next row blocks with cp.async while they transform
// the current one.
#include "vc_prep_common.cuh"

namespace vc {
namespace {

// ---------------------------------------------------------------------------------------
// RoPE tables: per axis a, entry [pos][i] = (cos, sin)(pos * theta^(-2 i / d_a)), evaluated
// in double and rounded once to fp32.
__global__ void rope_table_kernel(float2* tab, RopeDesc rd, double theta) {
  int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= rd.entries) return;
  int a = e >= rd.off[2] ? 2 : (e >= rd.off[1] ? 1 : 0);
  int r = e - rd.off[a];
  int pos = r / rd.pairs[a];
  int i = r - pos * rd.pairs[a];
  double freq = pow(theta, -2.0 * (double)i / (double)(2 * rd.pairs[a]));
  double phi = (double)pos * freq;
  const double c = cos(phi), sn = sin(phi);
  tab[e] = make_float2((float)c, (float)sn);
  // second table: the rotation folded into the first Hadamard level, u = x0 (c + s) + x1 (c - s),
  // v = x0 (c - s) - x1 (c + s), each coefficient rounded once
  tab[rd.entries + e] = make_float2((float)(c + sn), (float)(c - sn));
}

// ---------------------------------------------------------------------------------------
// Persistent, pipelined passes.  Every pass is a loop over work items (tensor, head, block of
// 128 rows); a CTA takes items blockIdx.x, blockIdx.x + gridDim.x, ...  The 16-byte chunks of
// the NEXT items are already on their way into a ring of shared-memory stages (cp.async, no
// registers held for bytes in flight) while the current item is transformed, so the load
// latency of a block hides behind the arithmetic of the blocks before it.  In the K column sums
// a thread fetches exactly the chunks it will read itself and in the Q/K pass a warp fetches
// exactly the rows it will transform, so those passes need no CTA-wide barrier for the data;
// V is staged as a tile because its codes leave channel-major.
// (One bulk-async copy per gathered row was tried instead of cp.async: 128 small copies per
// block kept the copy engine, not HBM, busy.)
constexpr int kThreads = 256;      // threads of the column-sum and V passes
constexpr int kRowThreads = 128;   // rows of a Q/K item (threads of the pass = rows x threads per row)
#ifndef VC_PREP_TPR
#define VC_PREP_TPR 2
#endif
#ifndef VC_PREP_TPR_FAST
#define VC_PREP_TPR_FAST VC_PREP_TPR      // threads per row of the packed row transform
#endif

template <int D> struct Geo {
  static constexpr int pitch = 2 * D + 16;          // row pitch of the thread-per-row layout
  static constexpr int stage_bytes = kBlock * pitch;
};

// Items are numbered block-fastest, then head, then tensor.  A CTA visits items blockIdx.x + k *
// gridDim.x: the position is divided out once and then advanced by the grid stride with carries
// (the divisions are not free at 64 elements per thread and item).
struct Cursor {
  int blk, hh, z;            // block, head within the launch's group, tensor
};
struct CursorStep {
  int dblk, dhh;             // gridDim.x = dhh * nb + dblk
};
__device__ __forceinline__ Cursor cursor_at(int item, int nb, int nh) {
  Cursor c;
  c.blk = item % nb;
  const int r = item / nb;
  c.hh = r % nh;
  c.z = r / nh;
  return c;
}
__device__ __forceinline__ CursorStep cursor_step(int nb) {
  CursorStep s;
  s.dhh = (int)gridDim.x / nb;
  s.dblk = (int)gridDim.x - s.dhh * nb;
  return s;
}
__device__ __forceinline__ void advance(Cursor& c, const CursorStep& s, int nb, int nh) {
  c.blk += s.dblk;
  c.hh += s.dhh;
  if (c.blk >= nb) { c.blk -= nb; ++c.hh; }
  while (c.hh >= nh) { c.hh -= nh; ++c.z; }      // at most once unless the launch is tiny
}
// Start of head bh in an input tensor, in bytes (bh = b * H + h, general strides).
__device__ __forceinline__ int64_t head_offset_bytes(const PrepArgs& a, int bh) {
  const int b = (int)div40((unsigned)bh, a.mul_H), h = bh - b * a.H;
  return 2 * (b * a.stride_b + h * a.stride_h);
}

// ---------------------------------------------------------------------------------------
// K column sums after RoPE (the channel mean of Sec. 3.4 is taken after the rotation).  A lane
// owns 8 consecutive channels of D/16 rows, so a column's partial sums meet by xor-shuffles.
// A RoPE table entry: from the copy in shared memory (address in the shared window) when there
// is one, else from global memory.
struct RopeTab {
  uint32_t saddr;            // 0: no copy in shared memory
  const float2* g;
};
__device__ __forceinline__ float2 rope_entry_s(uint32_t saddr, int e) {
  float2 r;
  asm("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(r.x), "=f"(r.y) : "r"(saddr + 8u * (uint32_t)e));
  return r;
}
__device__ __forceinline__ float2 rope_entry(const RopeTab& t, int e) {
  return t.saddr ? rope_entry_s(t.saddr, e) : __ldg(t.g + e);
}

struct PairSlots {          // the 4 channel pairs a lane owns: axis and table slot of each
  int axis[4], idx[4], stride[4];
};
__device__ __forceinline__ PairSlots pair_slots(const RopeDesc& rd, int first_pair) {
  PairSlots ps;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int p = first_pair + j;
    const int ax = p >= rd.pair_start[2] ? 2 : (p >= rd.pair_start[1] ? 1 : 0);
    ps.axis[j] = ax;
    ps.idx[j] = rd.off[ax] + (p - rd.pair_start[ax]);
    ps.stride[j] = rd.pairs[ax];
  }
  return ps;
}

template <int D>
__device__ __forceinline__ void k_colsum_item(const PrepArgs& a, const unsigned char* stage, float* red, const RopeTab& tab,
                                              const PairSlots& ps, int bh, int blk) {
  constexpr int LPR = D / 8;         // lanes per row
  constexpr int RPL = LPR / 2;       // rows per lane (a warp covers 16 rows)
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int lr = lane % LPR, hb = lane / LPR;
  const bool do_rope = a.flags & VC_FLAG_ROPE;
  // grid position of the lane's first row; the following rows advance x with carry
  int tt, ty, tx;
  grid_pos(a.rd, blk * kBlock + 16 * warp + RPL * hb, tt, ty, tx);
  float s[8];
#pragma unroll
  for (int c = 0; c < 8; ++c) s[c] = 0.f;
  const int t0 = blk * kBlock + 16 * warp + RPL * hb;
  const int n_rows = min(RPL, a.N - t0);           // rows of a lane ascend: the rest is padding
  if (do_rope && tab.saddr) {
    // The rotation is accumulated directly (four FMAs per channel pair and row).  The lane's four
    // table addresses follow its rows: x advances by one per row, so the entries of the pairs on
    // the x axis move by one table row and the others stay; a row that wraps x recomputes them.
    // The coefficients of the pairs on the t and y axes are the same for all of a lane's rows
    // unless x wraps, so they stay in registers; only lanes whose pairs lie on the x axis reload
    // per row (a predicated load: the other lanes take no shared-memory bandwidth).
    uint32_t ad[4], inc[4];
    float cc[4], ss[4];
    auto locate = [&]() {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int pos = ps.axis[j] == 0 ? tt : (ps.axis[j] == 1 ? ty : tx);
        ad[j] = tab.saddr + 8u * (uint32_t)(ps.idx[j] + pos * ps.stride[j]);
        asm("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(cc[j]), "=f"(ss[j]) : "r"(ad[j]));
      }
    };
#pragma unroll
    for (int j = 0; j < 4; ++j) inc[j] = ps.axis[j] == 2 ? 8u * (uint32_t)ps.stride[j] : 0u;
    locate();
#pragma unroll
    for (int i = 0; i < RPL; ++i) {
      if (i >= n_rows) break;
      const uint4 raw = *reinterpret_cast<const uint4*>(stage + (i * kThreads + tid) * 16);   // the chunk this thread fetched
      const unsigned int w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float x0 = __uint_as_float(w[j] << 16), x1 = __uint_as_float(w[j] & 0xffff0000u);
        s[2 * j] = fmaf(-x1, ss[j], fmaf(x0, cc[j], s[2 * j]));
        s[2 * j + 1] = fmaf(x1, cc[j], fmaf(x0, ss[j], s[2 * j + 1]));
      }
      if (i + 1 < RPL) {
        if (++tx == a.rd.grid_w) {
          tx = 0;
          if (++ty == a.rd.grid_h) { ty = 0; ++tt; }
          locate();
        } else {
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            if (inc[j]) {
              ad[j] += inc[j];
              asm("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(cc[j]), "=f"(ss[j]) : "r"(ad[j]));
            }
          }
        }
      }
    }
  } else {
#pragma unroll
    for (int i = 0; i < RPL; ++i) {
      if (i >= n_rows) break;
      const uint4 raw = *reinterpret_cast<const uint4*>(stage + (i * kThreads + tid) * 16);   // the chunk this thread fetched
      const unsigned int w[4] = {raw.x, raw.y, raw.z, raw.w};
      float x[8];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        x[2 * j] = __uint_as_float(w[j] << 16);
        x[2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
      }
      if (do_rope) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int pos = ps.axis[j] == 0 ? tt : (ps.axis[j] == 1 ? ty : tx);
          const float2 cs = rope_entry(tab, ps.idx[j] + pos * ps.stride[j]);
          const float x0 = x[2 * j], x1 = x[2 * j + 1];
          x[2 * j] = x0 * cs.x - x1 * cs.y;
          x[2 * j + 1] = x0 * cs.y + x1 * cs.x;
        }
        if (++tx == a.rd.grid_w) { tx = 0; if (++ty == a.rd.grid_h) { ty = 0; ++tt; } }
      }
#pragma unroll
      for (int c = 0; c < 8; ++c) s[c] += x[c];
    }
  }
#pragma unroll
  for (int c = 0; c < 8; ++c) {
#pragma unroll
    for (int m = LPR; m < 32; m <<= 1) s[c] += __shfl_xor_sync(0xffffffffu, s[c], m);
  }
  __syncthreads();                           // the previous item's reads of `red` are done
  if (hb == 0) {
#pragma unroll
    for (int c = 0; c < 8; ++c) red[warp * D + 8 * lr + c] = s[c];
  }
  __syncthreads();
  if (tid < D) {
    float t = 0.f;
#pragma unroll
    for (int w8 = 0; w8 < 8; ++w8) t += red[w8 * D + tid];
    a.k_part[((size_t)bh * a.nb + blk) * D + tid] = t;
  }
}

// ---------------------------------------------------------------------------------------
// Q / K, one row per thread.  All D channels of a row sit in the registers of one thread, so
// the Hadamard rotation is D/2 * log2 D register butterflies with no shuffle, RoPE pairs and
// NVFP4 groups are thread-local, and a row's codes leave as 16-byte stores.
enum { kStageAmax = 1, kStageQuant8 = 2, kStageQuant4 = 3, kStageQuant8I = 4 };   // 8I: INT8 codes (VC_FLAG_INT8_QK)

template <int D> struct RopeSplit;          // pair boundaries of the default channel split
template <> struct RopeSplit<128> { static constexpr int p1 = 22, p2 = 43; };   // 44 / 42 / 42
template <> struct RopeSplit<64> { static constexpr int p1 = 12, p2 = 22; };    // 24 / 20 / 20

// Reads the thread's row out of the stage, releases the stage, then transforms the row.
// `red` is [2][4] floats and `kmean_s` [D] floats of compute-warp scratch.
// Q and K run through one copy of the row body (TENSOR is a run-time argument): the unrolled body
// is tens of KB of code, and two copies of it thrash the instruction cache.
//
// TPR = threads per row.  With TPR = 1 a thread holds all D channels of its row.  With TPR = 2 the
// lanes 0..15 of a warp hold channels [0, D/2) of 16 rows and the lanes 16..31 channels [D/2, D)
// of the same rows: half the registers per thread, so twice the warps per SM; the last Hadamard
// level crosses the two halves with one shuffle per value.  RoPE pairs and NVFP4 groups stay
// thread-local either way.
template <int TPR> __device__ __forceinline__ int qk_row_of(int tid) {
  return TPR == 1 ? tid : (TPR == 2 ? 16 * (tid >> 5) + (tid & 15) : 8 * (tid >> 5) + (tid & 7));
}
template <int TPR> __device__ __forceinline__ int qk_part_of(int tid) {
  return TPR == 1 ? 0 : (TPR == 2 ? (tid >> 4) & 1 : (tid >> 3) & 3);
}

template <int D> __device__ __forceinline__ constexpr int rope_axis_of(int p) {
  return p < RopeSplit<D>::p1 ? 0 : (p < RopeSplit<D>::p2 ? 1 : 2);
}

template <int D, int STAGE, int TPR>
__device__ __forceinline__ void qk_row_item(const PrepArgs& a, const int TENSOR /*0 = Q, 1 = K*/, const unsigned char* stage,
                                            unsigned char* out_tile, float* red, float* kmean_s, const RopeTab& tab, int bh,
                                            int blk, int iter, bool new_head, int src_row) {
  constexpr int C = D / TPR;                       // channels per thread
  constexpr int NT = kRowThreads * TPR;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int row = qk_row_of<TPR>(tid), part = qk_part_of<TPR>(tid);
  const bool do_rope = a.flags & VC_FLAG_ROPE;
  const bool do_had = a.flags & VC_FLAG_HADAMARD;
  const bool center = TENSOR == 1 && (a.flags & VC_FLAG_K_SMOOTH);
  const bool valid = src_row >= 0;               // src_row: the input row behind this thread's row
  const int src = valid ? src_row : 0;           // (RoPE acts at the source position)
  // (a row without a source reads what the stage holds and is zeroed below)
  uint4 raw[C / 8];
#pragma unroll
  for (int i = 0; i < C / 8; ++i) raw[i] = *reinterpret_cast<const uint4*>(stage + row * Geo<D>::pitch + part * (2 * C) + 16 * i);
  if (center && new_head) {
    __syncthreads();                               // everyone is done with the previous head's mean
    for (int c = tid; c < D; c += NT) kmean_s[c] = a.k_mean[(size_t)bh * D + c];
    __syncthreads();
  }

  float x[C];
#pragma unroll
  for (int i = 0; i < C / 8; ++i) {
    const unsigned int w[4] = {raw[i].x, raw[i].y, raw[i].z, raw[i].w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      x[8 * i + 2 * j] = __uint_as_float(w[j] << 16);
      x[8 * i + 2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
    }
  }
  if (!valid) {
#pragma unroll
    for (int c = 0; c < C; ++c) x[c] = 0.f;
  }
  if (do_rope && valid) {
    int tt, ty, tx;
    grid_pos(a.rd, src, tt, ty, tx);
    // entry of pair p of axis ax: off[ax] + pos[ax] * pairs[ax] + (p - pair_start[ax])
    const int e[3] = {a.rd.off[0] + tt * a.rd.pairs[0] - a.rd.pair_start[0],
                      a.rd.off[1] + ty * a.rd.pairs[1] - a.rd.pair_start[1],
                      a.rd.off[2] + tx * a.rd.pairs[2] - a.rd.pair_start[2]};
    const int p0 = part * (C / 2);               // first pair of this thread
    if (a.rope_default && tab.saddr) {
      // compile-time pair boundaries: the axis of local pair i is known for either part, so the
      // table base of each (axis in part 0, axis in part 1) combination is selected once per row
      int base[3][3];
#pragma unroll
      for (int a0 = 0; a0 < 3; ++a0)
#pragma unroll
        for (int a1 = 0; a1 < 3; ++a1) base[a0][a1] = (part ? e[a1] : e[a0]) + p0;
#pragma unroll
      for (int i = 0; i < C / 2; ++i) {
        const float2 cs = rope_entry_s(tab.saddr, base[rope_axis_of<D>(i)][rope_axis_of<D>(TPR == 1 ? i : C / 2 + i)] + i);
        const float x0 = x[2 * i], x1 = x[2 * i + 1];
        x[2 * i] = x0 * cs.x - x1 * cs.y;
        x[2 * i + 1] = x0 * cs.y + x1 * cs.x;
      }
    } else {
#pragma unroll
      for (int i = 0; i < C / 2; ++i) {
        const int p = p0 + i;
        const int eb = p < a.rd.pair_start[1] ? e[0] : (p < a.rd.pair_start[2] ? e[1] : e[2]);
        const float2 cs = rope_entry(tab, eb + p);
        const float x0 = x[2 * i], x1 = x[2 * i + 1];
        x[2 * i] = x0 * cs.x - x1 * cs.y;
        x[2 * i + 1] = x0 * cs.y + x1 * cs.x;
      }
    }
  }
  if (center && valid) {
    const float4* km = reinterpret_cast<const float4*>(kmean_s + part * C);
#pragma unroll
    for (int c4 = 0; c4 < C / 4; ++c4) {
      const float4 m = km[c4];
      x[4 * c4] -= m.x; x[4 * c4 + 1] -= m.y; x[4 * c4 + 2] -= m.z; x[4 * c4 + 3] -= m.w;
    }
  }
  if (do_had) {
#pragma unroll
    for (int sft = 1; sft < C; sft <<= 1) {
#pragma unroll
      for (int c = 0; c < C; ++c) {
        if (!(c & sft)) {
          const float u = x[c], v = x[c | sft];
          x[c] = u + v;
          x[c | sft] = u - v;
        }
      }
    }
    if constexpr (TPR == 2) {
      // the level that pairs channel c with c + D/2: the lower half takes mine + theirs, the upper
      // half theirs - mine (one fused multiply-add with +-1, exact)
      const float sgn = part ? -1.0f : 1.0f;
#pragma unroll
      for (int c = 0; c < C; ++c) x[c] = fmaf(x[c], sgn, __shfl_xor_sync(0xffffffffu, x[c], 16));
    }
  }
  const float rs = do_had ? (D == 128 ? 0.08838834764831845f : 0.125f) : 1.0f;   // 1/sqrt(D)

  float amax = 0.f;
  if constexpr (STAGE != kStageQuant4) {
    float m0 = 0.f, m1 = 0.f;
#pragma unroll
    for (int c = 0; c < C; c += 4) {
      m0 = max3(m0, fabsf(x[c]), fabsf(x[c + 1]));
      m1 = max3(m1, fabsf(x[c + 2]), fabsf(x[c + 3]));
    }
    amax = warp_max(fmaxf(m0, m1) * rs);        // max and the (positive) scale commute exactly
    float* rbuf = red + 8 * (iter & 1);         // alternate buffers: one barrier per item suffices
    if (lane == 0) rbuf[warp] = amax;
    __syncthreads();
    amax = fmaxf(fmaxf(rbuf[0], rbuf[1]), fmaxf(rbuf[2], rbuf[3]));
    if constexpr (TPR == 2) amax = fmaxf(amax, fmaxf(fmaxf(rbuf[4], rbuf[5]), fmaxf(rbuf[6], rbuf[7])));
  }
  if constexpr (STAGE == kStageAmax) {
    if (tid == 0) atomicMax(&a.qk_amax[TENSOR * a.BH + bh], __float_as_uint(amax));
    return;
  }
  const size_t row_g = (size_t)bh * a.n_pad + (size_t)blk * kBlock + row;

  if constexpr (STAGE == kStageQuant8 || STAGE == kStageQuant8I) {
    // E4M3 codes (top value 448), or INT8 codes (top value 127; the INT8 Q K^T of Fig. 3)
    constexpr bool int8 = STAGE == kStageQuant8I;
    const float top = int8 ? 127.0f : 448.0f;
    const float inv = amax > 0.f ? top / amax : 0.f;
    if (tid == 0) (TENSOR == 0 ? a.q_scale : a.k_scale)[(size_t)bh * a.nb + blk] = amax > 0.f ? amax / top : 1.0f;
    // codes go to the swizzled output tile; the CTA copies it out with coalesced stores
    constexpr int CPR = D / 16;
    uint4* dst = reinterpret_cast<uint4*>(out_tile + row * D);
    const int sw = (row / (8 / CPR)) & (CPR - 1);
#pragma unroll
    for (int i = 0; i < C / 16; ++i) {
      unsigned int w[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int c = 16 * i + 4 * j;
        if constexpr (int8) {
          // |y| <= 127: adding 1.5 * 2^23 rounds y to the nearest even integer into the low mantissa
          // bits, two's complement for negative values; the low bytes are the codes
          const unsigned int r0 = __float_as_uint(((x[c] * rs) * inv) + 12582912.0f), r1 = __float_as_uint(((x[c + 1] * rs) * inv) + 12582912.0f);
          const unsigned int r2 = __float_as_uint(((x[c + 2] * rs) * inv) + 12582912.0f), r3 = __float_as_uint(((x[c + 3] * rs) * inv) + 12582912.0f);
          w[j] = __byte_perm(__byte_perm(r0, r1, 0x0040), __byte_perm(r2, r3, 0x0040), 0x5410);
        } else {
          const unsigned int lo = __nv_cvt_float2_to_fp8x2(make_float2((x[c] * rs) * inv, (x[c + 1] * rs) * inv), __NV_SATFINITE, __NV_E4M3);
          const unsigned int hi = __nv_cvt_float2_to_fp8x2(make_float2((x[c + 2] * rs) * inv, (x[c + 3] * rs) * inv), __NV_SATFINITE, __NV_E4M3);
          w[j] = lo | (hi << 16);
        }
      }
      dst[(part * (C / 16) + i) ^ sw] = make_uint4(w[0], w[1], w[2], w[3]);
    }
  }

  if constexpr (STAGE == kStageQuant4) {
    // NVFP4: outer scale g per (b, h), microscale per token per 16 channels
    const float g = (TENSOR == 0 ? a.q_scale : a.k_scale)[bh];
    const float inv6 = 1.0f / (6.0f * g);
    constexpr int MB = C / 16;                   // microscale bytes of this thread
    unsigned int codes[C / 8], micro[(MB + 3) / 4];
#pragma unroll
    for (int i = 0; i < (MB + 3) / 4; ++i) micro[i] = 0;
#pragma unroll
    for (int gq = 0; gq < C / 16; ++gq) {
      float m = 0.f;
#pragma unroll
      for (int c = 0; c < 16; ++c) { x[16 * gq + c] *= rs; m = fmaxf(m, fabsf(x[16 * gq + c])); }
      const unsigned int sb = __nv_cvt_float_to_fp8(m * inv6, __NV_SATFINITE, __NV_E4M3);
      const float sdec = e4m3_to_float(sb);
      const float rcp = sdec > 0.f ? 1.0f / (g * sdec) : 0.f;
      micro[gq / 4] |= sb << (8 * (gq & 3));
#pragma unroll
      for (int wi = 0; wi < 2; ++wi) {
        unsigned int word = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int c = 16 * gq + 8 * wi + 2 * j;
          const unsigned int two = __nv_cvt_float2_to_fp4x2(make_float2(x[c] * rcp, x[c + 1] * rcp), __NV_E2M1, cudaRoundNearest);
          word |= (two & 0xffu) << (8 * j);
        }
        codes[2 * gq + wi] = sdec > 0.f ? word : 0u;
      }
    }
    constexpr int CPR = D / 32;
    uint4* dst = reinterpret_cast<uint4*>(out_tile + row * (D / 2));
    const int sw = (row / (8 / CPR)) & (CPR - 1);
#pragma unroll
    for (int i = 0; i < C / 32; ++i) dst[(part * (C / 32) + i) ^ sw] = make_uint4(codes[4 * i], codes[4 * i + 1], codes[4 * i + 2], codes[4 * i + 3]);
    uint8_t* mrow = (TENSOR == 0 ? a.q_micro : a.k_micro) + row_g * (D / 16) + part * MB;
    if constexpr (MB % 4 == 0) {
#pragma unroll
      for (int i = 0; i < MB / 4; ++i) reinterpret_cast<unsigned int*>(mrow)[i] = micro[i];
    } else {
      static_assert(MB == 2, "microscale bytes per thread");
      *reinterpret_cast<unsigned short*>(mrow) = (unsigned short)micro[0];
    }
  }
}

// ---------------------------------------------------------------------------------------
// The same row transform with fewer instructions, for the standard configuration (RoPE with the
// default channel split and the table in shared memory, Hadamard on; K smoothing either way):
//  * rotation, centering and the first Hadamard level are one step per channel pair: with
//    (A, B) = (c + s, c - s) from the folded table and (m+, m-) = (m0 + m1, m0 - m1) of the mean,
//    u = x0 A + x1 B - m+  and  v = x0 B - x1 A - m-  are the level-1 outputs (4 FMAs per pair);
//  * a pair lives in one 64-bit register and the other levels, the cross-lane level and the scale
//    multiply are packed two-lane FP32 instructions (add / sub / fma / mul .f32x2: the same FP32
//    operation per lane, one instruction issued for two);
//  * at 8 bits 1 / sqrt(D) and the quantization scale are one factor.
// The 4-bit head-maximum and NVFP4 stages run on the same transform.
// `kmean_pm` holds (m+, m-) per pair, zeros while Q rows or unsmoothed K rows are processed.
template <int D, int STAGE, int TPR>
__device__ __forceinline__ void qk_row_item_fast(const PrepArgs& a, const int TENSOR, const unsigned char* stage,
                                                 unsigned char* out_tile, float* red, float* kmean_pm, uint32_t tab_saddr,
                                                 int bh, int blk, int iter, bool new_head, int src_row) {
  constexpr int C = D / TPR, P = C / 2;            // channels and pairs per thread
  constexpr int NT = kRowThreads * TPR;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int row = qk_row_of<TPR>(tid), part = qk_part_of<TPR>(tid);
  const bool valid = src_row >= 0;
  const int src = valid ? src_row : 0;
  uint4 raw[C / 8];
#pragma unroll
  for (int i = 0; i < C / 8; ++i) raw[i] = *reinterpret_cast<const uint4*>(stage + row * Geo<D>::pitch + part * (2 * C) + 16 * i);
  if (TENSOR == 1 && (a.flags & VC_FLAG_K_SMOOTH) && new_head) {
    __syncthreads();                               // everyone is done with the previous head's mean
    for (int pr = tid; pr < D / 2; pr += NT) {
      const float2 m = *reinterpret_cast<const float2*>(a.k_mean + (size_t)bh * D + 2 * pr);
      *reinterpret_cast<float2*>(kmean_pm + 2 * pr) = make_float2(m.x + m.y, m.x - m.y);
    }
    __syncthreads();
  }
  int tt, ty, tx;
  grid_pos(a.rd, src, tt, ty, tx);
  const int e[3] = {a.rd.off[0] + tt * a.rd.pairs[0] - a.rd.pair_start[0],
                    a.rd.off[1] + ty * a.rd.pairs[1] - a.rd.pair_start[1],
                    a.rd.off[2] + tx * a.rd.pairs[2] - a.rd.pair_start[2]};
  const int p0 = part * P;
  // byte address of pair i's entry = base of its axis + 8 i (the axis of local pair i is known at
  // compile time for either part: one base per combination, selected once per row)
  // (written as a selection per pair; identical selections fold into one value per combination)
  auto base_of = [&](int i) -> uint32_t {          // i is a compile-time constant after unrolling
    int ee;
    if constexpr (TPR == 1) ee = e[rope_axis_of<D>(i)];
    else if constexpr (TPR == 2) ee = part ? e[rope_axis_of<D>(P + i)] : e[rope_axis_of<D>(i)];
    else ee = part == 0 ? e[rope_axis_of<D>(i)] : (part == 1 ? e[rope_axis_of<D>(P + i)] : (part == 2 ? e[rope_axis_of<D>(2 * P + i)] : e[rope_axis_of<D>(3 * P + i)]));
    return tab_saddr + 8u * (uint32_t)(ee + p0);
  };
  const float4* km = reinterpret_cast<const float4*>(kmean_pm + part * C);

  uint64_t X[P];
#pragma unroll
  for (int i = 0; i < P; i += 2) {
    const float4 m = km[i / 2];                    // (m+, m-) of pairs i and i + 1
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int ii = i + k;
      const unsigned int w = ii % 4 == 0 ? raw[ii / 4].x : (ii % 4 == 1 ? raw[ii / 4].y : (ii % 4 == 2 ? raw[ii / 4].z : raw[ii / 4].w));
      const float x0 = __uint_as_float(w << 16), x1 = __uint_as_float(w & 0xffff0000u);
      float A, B;
      asm("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(A), "=f"(B)
          : "r"(base_of(ii) + 8u * ii));
      const float mp = k == 0 ? m.x : m.z, mm = k == 0 ? m.y : m.w;
      const float u = fmaf(x0, A, fmaf(x1, B, -mp));
      const float v = fmaf(x0, B, fmaf(-x1, A, -mm));
      X[ii] = pack_f32x2(u, v);
    }
  }
  if (!valid) {                                    // a padding row: zeros (codes 0, no part in the maximum)
#pragma unroll
    for (int i = 0; i < P; ++i) X[i] = 0ull;
  }
  // Hadamard levels 2 .. C/2 on whole pairs
#pragma unroll
  for (int h = 1; h < P; h <<= 1) {
#pragma unroll
    for (int i = 0; i < P; ++i) {
      if (!(i & h)) {
        const uint64_t U = X[i], V = X[i | h];
        X[i] = add2(U, V);
        X[i | h] = sub2(U, V);
      }
    }
  }
  if constexpr (TPR >= 2) {
    // the levels that pair channels across the threads of a row (distance C, then 2 C with four
    // threads per row): the lower part takes mine + theirs, the upper part theirs - mine
#pragma unroll
    for (int lv = 0; lv < (TPR == 2 ? 1 : 2); ++lv) {
      const int mask = TPR == 2 ? 16 : (lv == 0 ? 8 : 16);
      const float sg = ((part >> lv) & 1) ? -1.0f : 1.0f;
      const uint64_t SG = pack_f32x2(sg, sg);
#pragma unroll
      for (int i = 0; i < P; ++i) {
        float lo, hi;
        unpack2(X[i], lo, hi);
        const float olo = __shfl_xor_sync(0xffffffffu, lo, mask), ohi = __shfl_xor_sync(0xffffffffu, hi, mask);
        X[i] = fma2(X[i], SG, pack_f32x2(olo, ohi));
      }
    }
  }
  constexpr float rs = D == 128 ? 0.08838834764831845f : 0.125f;   // 1/sqrt(D)

  float amax = 0.f;
  if constexpr (STAGE != kStageQuant4) {
    float m0 = 0.f, m1 = 0.f;
#pragma unroll
    for (int i = 0; i < P; i += 2) {
      float a0, a1, b0, b1;
      unpack2(X[i], a0, a1);
      unpack2(X[i + 1], b0, b1);
      m0 = max3(m0, fabsf(a0), fabsf(a1));
      m1 = max3(m1, fabsf(b0), fabsf(b1));
    }
    amax = warp_max(fmaxf(m0, m1) * rs);           // max and the (positive) scale commute exactly
    float* rbuf = red + 16 * (iter & 1);           // alternate buffers: one barrier per item suffices
    if (lane == 0) rbuf[warp] = amax;
    __syncthreads();
    amax = fmaxf(fmaxf(rbuf[0], rbuf[1]), fmaxf(rbuf[2], rbuf[3]));
    if constexpr (TPR >= 2) amax = fmaxf(amax, fmaxf(fmaxf(rbuf[4], rbuf[5]), fmaxf(rbuf[6], rbuf[7])));
    if constexpr (TPR == 4) {
      amax = fmaxf(amax, fmaxf(fmaxf(rbuf[8], rbuf[9]), fmaxf(rbuf[10], rbuf[11])));
      amax = fmaxf(amax, fmaxf(fmaxf(rbuf[12], rbuf[13]), fmaxf(rbuf[14], rbuf[15])));
    }
  }
  if constexpr (STAGE == kStageAmax) {
    if (tid == 0) atomicMax(&a.qk_amax[TENSOR * a.BH + bh], __float_as_uint(amax));
    return;
  }
  if constexpr (STAGE == kStageQuant4) {
    // NVFP4: outer scale g per (b, h), microscale per token per 16 channels (the arithmetic of the
    // general row body: y = x / sqrt(D), then y / (g * microscale), each rounded once)
    const float g = (TENSOR == 0 ? a.q_scale : a.k_scale)[bh];
    const float inv6 = 1.0f / (6.0f * g);
    const uint64_t RS = pack_f32x2(rs, rs);
    constexpr int MB = C / 16;                     // microscale bytes of this thread
    unsigned int codes[C / 8], micro[(MB + 3) / 4];
#pragma unroll
    for (int i = 0; i < (MB + 3) / 4; ++i) micro[i] = 0;
#pragma unroll
    for (int gq = 0; gq < C / 16; ++gq) {
      float m0 = 0.f, m1 = 0.f;
#pragma unroll
      for (int i = 0; i < 8; i += 2) {
        float a0, a1, b0, b1;
        X[8 * gq + i] = mul2(X[8 * gq + i], RS);
        X[8 * gq + i + 1] = mul2(X[8 * gq + i + 1], RS);
        unpack2(X[8 * gq + i], a0, a1);
        unpack2(X[8 * gq + i + 1], b0, b1);
        m0 = max3(m0, fabsf(a0), fabsf(a1));
        m1 = max3(m1, fabsf(b0), fabsf(b1));
      }
      const float m = fmaxf(m0, m1);
      const unsigned int sb = __nv_cvt_float_to_fp8(m * inv6, __NV_SATFINITE, __NV_E4M3);
      const float sdec = e4m3_to_float(sb);
      const float rcp = sdec > 0.f ? 1.0f / (g * sdec) : 0.f;
      const uint64_t RC = pack_f32x2(rcp, rcp);
      micro[gq / 4] |= sb << (8 * (gq & 3));
#pragma unroll
      for (int wi = 0; wi < 2; ++wi) {
        unsigned int word = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          float y0, y1;
          unpack2(mul2(X[8 * gq + 4 * wi + j], RC), y0, y1);
          const unsigned int two = __nv_cvt_float2_to_fp4x2(make_float2(y0, y1), __NV_E2M1, cudaRoundNearest);
          word |= (two & 0xffu) << (8 * j);
        }
        codes[2 * gq + wi] = sdec > 0.f ? word : 0u;
      }
    }
    constexpr int CPR4 = D / 32;
    uint4* dst4 = reinterpret_cast<uint4*>(out_tile + row * (D / 2));
    const int sw4 = (row / (8 / CPR4)) & (CPR4 - 1);
#pragma unroll
    for (int i = 0; i < C / 32; ++i) dst4[(part * (C / 32) + i) ^ sw4] = make_uint4(codes[4 * i], codes[4 * i + 1], codes[4 * i + 2], codes[4 * i + 3]);
    const size_t row_g = (size_t)bh * a.n_pad + (size_t)blk * kBlock + row;
    uint8_t* mrow = (TENSOR == 0 ? a.q_micro : a.k_micro) + row_g * (D / 16) + part * MB;
    if constexpr (MB % 4 == 0) {
#pragma unroll
      for (int i = 0; i < MB / 4; ++i) reinterpret_cast<unsigned int*>(mrow)[i] = micro[i];
    } else {
      static_assert(MB == 2, "microscale bytes per thread");
      *reinterpret_cast<unsigned short*>(mrow) = (unsigned short)micro[0];
    }
    return;
  }

  constexpr bool int8 = STAGE == kStageQuant8I;
  const float top = int8 ? 127.0f : 448.0f;
  const float f = amax > 0.f ? rs * (top / amax) : 0.f;   // 1/sqrt(D) and 1/scale in one factor
  if (tid == 0) (TENSOR == 0 ? a.q_scale : a.k_scale)[(size_t)bh * a.nb + blk] = amax > 0.f ? amax / top : 1.0f;
  const uint64_t F = pack_f32x2(f, f);
  constexpr int CPR = D / 16;
  uint4* dst = reinterpret_cast<uint4*>(out_tile + row * D);
  const int sw = (row / (8 / CPR)) & (CPR - 1);
#pragma unroll
  for (int i = 0; i < C / 16; ++i) {
    unsigned int w[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int pi = 8 * i + 2 * j;                // pairs pi, pi + 1 = channels 16 i + 4 j .. + 3
      if constexpr (int8) {
        const uint64_t MG = pack_f32x2(12582912.0f, 12582912.0f);
        const uint64_t ra = fma2(X[pi], F, MG), rb = fma2(X[pi + 1], F, MG);
        w[j] = __byte_perm(__byte_perm((unsigned int)ra, (unsigned int)(ra >> 32), 0x0040),
                           __byte_perm((unsigned int)rb, (unsigned int)(rb >> 32), 0x0040), 0x5410);
      } else {
        float y0, y1, y2, y3;
        unpack2(mul2(X[pi], F), y0, y1);
        unpack2(mul2(X[pi + 1], F), y2, y3);
        const unsigned int lo = __nv_cvt_float2_to_fp8x2(make_float2(y0, y1), __NV_SATFINITE, __NV_E4M3);
        const unsigned int hi = __nv_cvt_float2_to_fp8x2(make_float2(y2, y3), __NV_SATFINITE, __NV_E4M3);
        w[j] = lo | (hi << 16);
      }
    }
    dst[(part * (C / 16) + i) ^ sw] = make_uint4(w[0], w[1], w[2], w[3]);
  }
}

// ---------------------------------------------------------------------------------------
// V.  A thread owns one channel pair and 128 / (256 / (D/2)) consecutive tokens of the gathered
// block, so block means and the channel-major (token-contiguous) code rows need no transposition.
enum { kVStats = 0, kVQuant8 = 1, kVQuant4 = 2, kVQuant4M = 3 };   // 4M: E2M1 under power-of-two factors per 32 tokens

// Statistics of a value block (launch 1b): block mean per channel (Eq. 4) and the block's
// max |v - mu|, folded into the head's per-channel maximum.  One pass over the thread's tokens
// collects the sum, the maximum and the minimum (the last two on the packed bf16 pairs as they
// are: max/min.bf16x2), one exchange combines the token groups, and
//     max_i |v_i - mu| = max(max_i v_i - mu, mu - min_i v_i)
// bit for bit, because the FP32 subtraction is monotonic.
template <int D, bool FULL>
__device__ __forceinline__ void v_stats_item(const PrepArgs& a, const unsigned char* stage, float* red, int bh, int blk) {
  constexpr int CP = D / 2, TG = kThreads / CP, TPG = kBlock / TG;
  const int tid = threadIdx.x;
  const int cp = tid % CP, tg = tid / CP;
  const int n_valid = FULL ? kBlock : min(kBlock, a.N - blk * kBlock);
  const unsigned char* mine = stage + tg * TPG * (2 * D) + 4 * cp;
  float s0 = 0.f, s1 = 0.f;
  __nv_bfloat162 mx = __halves2bfloat162(__ushort_as_bfloat16(0xff80), __ushort_as_bfloat16(0xff80));   // -inf
  __nv_bfloat162 mn = __halves2bfloat162(__ushort_as_bfloat16(0x7f80), __ushort_as_bfloat16(0x7f80));   // +inf
#pragma unroll
  for (int i = 0; i < TPG; ++i) {
    if (FULL || tg * TPG + i < n_valid) {
      const unsigned int w = *reinterpret_cast<const unsigned int*>(mine + i * (2 * D));
      s0 += __uint_as_float(w << 16);
      s1 += __uint_as_float(w & 0xffff0000u);
      const __nv_bfloat162 v = *reinterpret_cast<const __nv_bfloat162*>(&w);
      mx = __hmax2(mx, v);
      mn = __hmin2(mn, v);
    }
  }
  // red: [TG][D] sums, then [TG][CP] packed maxima, then [TG][CP] packed minima
  unsigned int* red_mx = reinterpret_cast<unsigned int*>(red + TG * D);
  unsigned int* red_mn = red_mx + TG * CP;
  *reinterpret_cast<float2*>(red + tg * D + 2 * cp) = make_float2(s0, s1);
  red_mx[tg * CP + cp] = *reinterpret_cast<unsigned int*>(&mx);
  red_mn[tg * CP + cp] = *reinterpret_cast<unsigned int*>(&mn);
  __syncthreads();                           // (the barrier at the top of the next item covers these reads)
  if (tg == 0) {
    s0 = 0.f; s1 = 0.f;
#pragma unroll
    for (int g = 0; g < TG; ++g) {
      const float2 p = *reinterpret_cast<const float2*>(red + g * D + 2 * cp);
      s0 += p.x; s1 += p.y;
      if (g > 0) {
        mx = __hmax2(mx, *reinterpret_cast<const __nv_bfloat162*>(&red_mx[g * CP + cp]));
        mn = __hmin2(mn, *reinterpret_cast<const __nv_bfloat162*>(&red_mn[g * CP + cp]));
      }
    }
    const bool smooth = a.flags & VC_FLAG_V_SMOOTH;
    const float mu0 = smooth ? s0 / (float)n_valid : 0.f, mu1 = smooth ? s1 / (float)n_valid : 0.f;
    const size_t mu_at = ((size_t)bh * a.nb + blk) * D + 2 * cp;
    *reinterpret_cast<float2*>(a.v_mu + mu_at) = make_float2(mu0, mu1);
    const float2 hi = __bfloat1622float2(mx), lo = __bfloat1622float2(mn);
    const float m0 = fmaxf(hi.x - mu0, mu0 - lo.x), m1 = fmaxf(hi.y - mu1, mu1 - lo.y);
    atomicMax(&a.v_amax[(size_t)bh * D + 2 * cp], __float_as_uint(m0));
    atomicMax(&a.v_amax[(size_t)bh * D + 2 * cp + 1], __float_as_uint(m1));
  }
}

// FULL: all 128 rows of the block exist (every block but a head's ragged last one): no row tests.
template <int D, int STAGE, bool FULL>
__device__ __forceinline__ void v_item(const PrepArgs& a, const unsigned char* stage, float* red, int bh, int blk,
                                       float2 mu_in, float2 am_in) {
  constexpr int CP = D / 2;             // channel pairs
  constexpr int TG = kThreads / CP;     // token groups
  constexpr int TPG = kBlock / TG;      // tokens per thread
  const int tid = threadIdx.x;
  const int cp = tid % CP, tg = tid / CP;
  const int n_valid = FULL ? kBlock : min(kBlock, a.N - blk * kBlock);
  float v0[TPG], v1[TPG];
  const unsigned char* mine = stage + tg * TPG * (2 * D) + 4 * cp;
#pragma unroll
  for (int i = 0; i < TPG; ++i) {
    const unsigned int w = (FULL || tg * TPG + i < n_valid) ? *reinterpret_cast<const unsigned int*>(mine + i * (2 * D)) : 0u;
    v0[i] = __uint_as_float(w << 16);
    v1[i] = __uint_as_float(w & 0xffff0000u);
  }
  const bool smooth = a.flags & VC_FLAG_V_SMOOTH;
  const size_t mu_at = ((size_t)bh * a.nb + blk) * D + 2 * cp;
  float mu0 = 0.f, mu1 = 0.f;

  // At 4 bits the values have no tensor-level scale, so nothing of a block's codes depends on
  // other blocks: the block mean is formed here, in the quantizing pass, and the statistics
  // launch is not needed.
  constexpr bool kFusedMean = STAGE == kVQuant4 || STAGE == kVQuant4M;
  static_assert(STAGE != kVStats, "the statistics stage has its own item function");
  if constexpr (kFusedMean) {
    __syncthreads();                         // the previous item's reads of `red` are done
    if (smooth) {
      float s0 = 0.f, s1 = 0.f;
#pragma unroll
      for (int i = 0; i < TPG; ++i) { s0 += v0[i]; s1 += v1[i]; }
      red[tg * D + 2 * cp] = s0;
      red[tg * D + 2 * cp + 1] = s1;
      __syncthreads();
      s0 = 0.f; s1 = 0.f;
#pragma unroll
      for (int g = 0; g < TG; ++g) { s0 += red[g * D + 2 * cp]; s1 += red[g * D + 2 * cp + 1]; }
      mu0 = s0 / (float)n_valid;
      mu1 = s1 / (float)n_valid;
      if constexpr (kFusedMean) {
        // at 4 bits the mean is stored as bf16 and added back unscaled (App. B): subtract exactly
        // that number, so that Eq. 6 restores what Eq. 4 removed
        mu0 = __bfloat162float(__float2bfloat16_rn(mu0));
        mu1 = __bfloat162float(__float2bfloat16_rn(mu1));
      }
      __syncthreads();
    }
  }
  if constexpr (!kFusedMean) {
    mu0 = mu_in.x;
    mu1 = mu_in.y;
  }
  float r0[TPG], r1[TPG];
#pragma unroll
  for (int i = 0; i < TPG; ++i) {
    const bool valid = FULL || tg * TPG + i < n_valid;
    r0[i] = valid ? v0[i] - mu0 : 0.f;
    r1[i] = valid ? v1[i] - mu1 : 0.f;
  }
  const size_t tok0 = (size_t)blk * kBlock + tg * TPG;

  if constexpr (STAGE == kVQuant8) {
    const float am0 = am_in.x, am1 = am_in.y;
    const float inv0 = am0 > 0.f ? 448.0f / am0 : 0.f, inv1 = am1 > 0.f ? 448.0f / am1 : 0.f;
    unsigned int w0[TPG / 4], w1[TPG / 4];
#pragma unroll
    for (int j = 0; j < TPG / 4; ++j) {
      unsigned int lo = __nv_cvt_float2_to_fp8x2(make_float2(r0[4 * j] * inv0, r0[4 * j + 1] * inv0), __NV_SATFINITE, __NV_E4M3);
      unsigned int hi = __nv_cvt_float2_to_fp8x2(make_float2(r0[4 * j + 2] * inv0, r0[4 * j + 3] * inv0), __NV_SATFINITE, __NV_E4M3);
      w0[j] = lo | (hi << 16);
      lo = __nv_cvt_float2_to_fp8x2(make_float2(r1[4 * j] * inv1, r1[4 * j + 1] * inv1), __NV_SATFINITE, __NV_E4M3);
      hi = __nv_cvt_float2_to_fp8x2(make_float2(r1[4 * j + 2] * inv1, r1[4 * j + 3] * inv1), __NV_SATFINITE, __NV_E4M3);
      w1[j] = lo | (hi << 16);
    }
    uint4* d0 = reinterpret_cast<uint4*>(a.v_codes + ((size_t)bh * D + 2 * cp) * a.n_pad + tok0);
    uint4* d1 = reinterpret_cast<uint4*>(a.v_codes + ((size_t)bh * D + 2 * cp + 1) * a.n_pad + tok0);
#pragma unroll
    for (int j = 0; j < TPG / 16; ++j) {
      d0[j] = make_uint4(w0[4 * j], w0[4 * j + 1], w0[4 * j + 2], w0[4 * j + 3]);
      d1[j] = make_uint4(w1[4 * j], w1[4 * j + 1], w1[4 * j + 2], w1[4 * j + 3]);
    }
    if (tg == 0) {   // block means stored divided by the value scale (App. B)
      const float a0 = mu0 * (am0 > 0.f ? inv0 : 1.0f), a1 = mu1 * (am1 > 0.f ? inv1 : 1.0f);
      *reinterpret_cast<__nv_bfloat162*>(a.v_means + mu_at) = __floats2bfloat162_rn(a0, a1);
    }
  }

  if constexpr (STAGE == kVQuant4) {
    // NVFP4 along tokens: one microscale per channel per 16 consecutive permuted tokens
    const float sixth = 1.0f / 6.0f;
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      const float* r = half == 0 ? r0 : r1;
      const int c = 2 * cp + half;
      unsigned int packed[TPG / 8];
      unsigned int micro = 0;
#pragma unroll
      for (int gq = 0; gq < TPG / 16; ++gq) {
        float m = 0.f;
#pragma unroll
        for (int i = 0; i < 16; ++i) m = fmaxf(m, fabsf(r[16 * gq + i]));
        const unsigned int sb = __nv_cvt_float_to_fp8(m * sixth, __NV_SATFINITE, __NV_E4M3);
        const float sdec = e4m3_to_float(sb);
        const float rcp = sdec > 0.f ? 1.0f / sdec : 0.f;
        micro |= sb << (8 * gq);
#pragma unroll
        for (int wi = 0; wi < 2; ++wi) {
          unsigned int word = 0;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int i = 16 * gq + 8 * wi + 2 * j;
            const unsigned int two = __nv_cvt_float2_to_fp4x2(make_float2(r[i] * rcp, r[i + 1] * rcp), __NV_E2M1, cudaRoundNearest);
            word |= (two & 0xffu) << (8 * j);
          }
          packed[2 * gq + wi] = sdec > 0.f ? word : 0u;
        }
      }
      uint8_t* d = a.v_codes + ((size_t)bh * D + c) * (a.n_pad / 2) + tok0 / 2;
      uint8_t* md = a.v_micro + ((size_t)bh * D + c) * (a.n_pad / 16) + tok0 / 16;
      if constexpr (TPG == 32) {
        *reinterpret_cast<uint4*>(d) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
        *reinterpret_cast<unsigned short*>(md) = (unsigned short)micro;
      } else {
        *reinterpret_cast<uint2*>(d) = make_uint2(packed[0], packed[1]);
        *md = (uint8_t)micro;
      }
    }
    if (tg == 0)
      *reinterpret_cast<__nv_bfloat162*>(a.v_means + mu_at) = __floats2bfloat162_rn(mu0, mu1);
  }

  if constexpr (STAGE == kVQuant4M) {
    // E2M1 under one power-of-two factor per channel per 32 consecutive permuted tokens (the
    // operand format of the FP8 x FP4 block-scaled product).  Factor 2^e with e the smallest
    // exponent that keeps the group maximum inside the E2M1 range: y = max / 6 (one division),
    // e = exponent(y), plus one unless y is a power of two.  Scaling by 2^-e is exact.
    float m0 = 0.f, m1 = 0.f;
#pragma unroll
    for (int i = 0; i < TPG; ++i) { m0 = fmaxf(m0, fabsf(r0[i])); m1 = fmaxf(m1, fabsf(r1[i])); }
    if constexpr (TPG == 16) {               // a group spans two threads (token groups 2g, 2g + 1)
      __syncthreads();                       // the previous item's reads of `red` are done
      red[tg * D + 2 * cp] = m0;
      red[tg * D + 2 * cp + 1] = m1;
      __syncthreads();
      m0 = fmaxf(m0, red[(tg ^ 1) * D + 2 * cp]);
      m1 = fmaxf(m1, red[(tg ^ 1) * D + 2 * cp + 1]);
    }
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      const float* r = half == 0 ? r0 : r1;
      const float m = half == 0 ? m0 : m1;
      const int c = 2 * cp + half;
      const unsigned int yb = __float_as_uint(__fdiv_rn(m, 6.0f));
      int code = (int)((yb >> 23) & 0xffu) + ((yb & 0x7fffffu) ? 1 : 0);     // e + 127
      code = m > 0.f ? min(max(code, 0), 254) : 0;
      const float rs = __uint_as_float((unsigned int)(254 - code) << 23);     // 2^-e
      unsigned int packed[TPG / 8];
#pragma unroll
      for (int wi = 0; wi < TPG / 8; ++wi) {
        unsigned int word = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int i = 8 * wi + 2 * j;
          const unsigned int two = __nv_cvt_float2_to_fp4x2(make_float2(r[i] * rs, r[i + 1] * rs), __NV_E2M1, cudaRoundNearest);
          word |= (two & 0xffu) << (8 * j);
        }
        packed[wi] = m > 0.f ? word : 0u;
      }
      uint8_t* d = a.v_codes + ((size_t)bh * D + c) * (a.n_pad / 2) + tok0 / 2;
      uint8_t* md = a.v_micro + ((size_t)bh * D + c) * (a.n_pad / 32) + tok0 / 32;
      if constexpr (TPG == 32) {
        *reinterpret_cast<uint4*>(d) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
        *md = (uint8_t)code;
      } else {
        *reinterpret_cast<uint2*>(d) = make_uint2(packed[0], packed[1]);
        if ((tg & 1) == 0) *md = (uint8_t)code;
      }
    }
    if (tg == 0)
      *reinterpret_cast<__nv_bfloat162*>(a.v_means + mu_at) = __floats2bfloat162_rn(mu0, mu1);
  }
}

// ---------------------------------------------------------------------------------------
// RoPE table -> shared memory (when it fits), once per CTA.
__device__ __forceinline__ RopeTab stage_rope_table(const PrepArgs& a, unsigned char* at, bool folded = false) {
  const float2* src = a.rope + (folded ? a.rd.entries : 0);
  RopeTab tab{0u, src};
  if ((a.flags & VC_FLAG_ROPE) && a.rope_in_smem) {
    float2* tab_s = reinterpret_cast<float2*>(at);
    for (int e = threadIdx.x; e < a.rd.entries; e += blockDim.x) tab_s[e] = __ldg(&src[e]);
    tab.saddr = smem_u32(at);
  }
  __syncthreads();
  return tab;
}

// Launch 1a: column sums of RoPE(K) per block (the channel mean is taken after the rotation).
// Shared memory: [2 stages x 32 KB][red: 8 D floats][RoPE table].
template <int D>
__global__ void __launch_bounds__(kThreads, 2) prep_kcolsum_kernel(const PrepArgs a, int n_items, int nh) {
  constexpr int LPR = D / 8, RPL = LPR / 2, kStage = kThreads * RPL * 16;
  extern __shared__ __align__(128) unsigned char smem[];
  float* red = reinterpret_cast<float*>(smem + 2 * kStage);
  const RopeTab tab = stage_rope_table(a, smem + 2 * kStage + 8 * D * 4);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int lr = lane % LPR, hb = lane / LPR;
  const PairSlots ps = pair_slots(a.rd, 4 * lr);
  const CursorStep step = cursor_step(a.nb);
  auto issue = [&](int item, const Cursor& c, int st) {
    if (item < n_items) {
      const char* base = reinterpret_cast<const char*>(a.k) + head_offset_bytes(a, a.bh0 + c.hh) + 16 * lr;
      const int t0 = c.blk * kBlock + 16 * warp + RPL * hb;
      unsigned char* dst = smem + st * kStage + tid * 16;
#pragma unroll
      for (int i = 0; i < RPL; ++i)
        if (t0 + i < a.N) cp_async16(dst + i * kThreads * 16, base + (int64_t)(t0 + i) * a.stride_n_bytes);
    }
    cp_async_commit();
  };
  Cursor cur = cursor_at(blockIdx.x, a.nb, nh), nxt = cur;
  advance(nxt, step, a.nb, nh);
  issue(blockIdx.x, cur, 0);
  int i = 0;
  for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++i) {
    issue(item + gridDim.x, nxt, (i + 1) & 1);
    cp_async_wait<1>();                       // this thread's chunks of item i have landed
    k_colsum_item<D>(a, smem + (i & 1) * kStage, red, tab, ps, a.bh0 + cur.hh, cur.blk);
    cur = nxt;
    advance(nxt, step, a.nb, nh);
  }
}

// V pass: STAGE = block means + residual amax (launch 1b) or quantization of the residual.
// Shared memory: [3 stages x (128 x 2 D)][red: 16 D floats][source rows: 2 x 128].
template <int D, int STAGE>
__global__ void __launch_bounds__(kThreads, 2) prep_v_kernel(const PrepArgs a, int n_items, int nh) {
  constexpr int LPR = D / 8, kStage = kBlock * 2 * D, NL = kBlock * LPR / kThreads;
  extern __shared__ __align__(128) unsigned char smem[];
  float* red = reinterpret_cast<float*>(smem + 3 * kStage);
  int* src_ring = reinterpret_cast<int*>(red + 16 * D);                // [2][128]
  const int tid = threadIdx.x;
  const CursorStep step = cursor_step(a.nb);
  // source row of row `tid` of an item (the gather by pi), -1 if there is none
  auto fetch = [&](int item, const Cursor& c) -> int {
    if (item >= n_items || tid >= kBlock) return -1;
    const int t = c.blk * kBlock + tid;
    if (t >= a.N) return -1;
    return a.perm ? min(max(__ldg(a.perm + (size_t)(a.bh0 + c.hh) * a.N + t), 0), a.N - 1) : t;   // clamped: never a bad address
  };
  auto issue = [&](int item, const Cursor& c, int st, const int* src) {
    if (item < n_items) {
      const char* base = reinterpret_cast<const char*>(a.v) + head_offset_bytes(a, a.bh0 + c.hh) + 16 * (tid % LPR);
      unsigned char* dst = smem + st * kStage + tid * 16;
#pragma unroll
      for (int k = 0; k < NL; ++k) {
        const int sr = src[tid / LPR + k * (kThreads / LPR)];
        if (sr >= 0) cp_async16(dst + k * kThreads * 16, base + (int64_t)sr * a.stride_n_bytes);
      }
    }
    cp_async_commit();
  };
  // per-item scalars of the quantizing stage, fetched one item ahead
  const int cp = tid % (D / 2);
  auto fetch_mu = [&](int item, const Cursor& c) -> float2 {
    if (STAGE == kVStats || STAGE == kVQuant4 || STAGE == kVQuant4M || item >= n_items) return make_float2(0.f, 0.f);
    return *reinterpret_cast<const float2*>(a.v_mu + ((size_t)(a.bh0 + c.hh) * a.nb + c.blk) * D + 2 * cp);
  };
  // cursors of items i, i+1, i+2 and i+4 of this CTA
  const int g = gridDim.x;
  Cursor c0 = cursor_at(blockIdx.x, a.nb, nh), c1 = c0;
  advance(c1, step, a.nb, nh);
  Cursor c2 = c1;
  advance(c2, step, a.nb, nh);
  Cursor c4 = c2;
  advance(c4, step, a.nb, nh);
  if (tid < kBlock) {
    src_ring[tid] = fetch(blockIdx.x, c0);
    src_ring[kBlock + tid] = fetch(blockIdx.x + g, c1);
  }
  __syncthreads();
  issue(blockIdx.x, c0, 0, src_ring);
  issue(blockIdx.x + g, c1, 1, src_ring + kBlock);
  __syncthreads();                            // the two slices have been read
  if (tid < kBlock) src_ring[tid] = fetch(blockIdx.x + 2 * g, c2);
  int nxt = fetch(blockIdx.x + 3 * g, c4);    // (c4 still stands at item 3 here)
  advance(c4, step, a.nb, nh);
  float2 mu = fetch_mu(blockIdx.x, c0), am = make_float2(0.f, 0.f);
  int i = 0, last_hh = -1;
  for (int item = blockIdx.x; item < n_items; item += g, ++i) {
    cp_async_wait<1>();                       // my chunks of item i have landed ...
    __syncthreads();                          // ... and everyone's; all are done with item i-1
    if (tid < kBlock) src_ring[((i + 1) & 1) * kBlock + tid] = nxt;     // source rows of item i+3
    nxt = fetch(item + 4 * g, c4);
    issue(item + 2 * g, c2, (i + 2) % 3, src_ring + (i & 1) * kBlock);
    const float2 mu_next = fetch_mu(item + g, c1);
    if (STAGE == kVQuant8 && c0.hh != last_hh) {
      const size_t at = (size_t)(a.bh0 + c0.hh) * D + 2 * cp;
      am = make_float2(__uint_as_float(a.v_amax[at]), __uint_as_float(a.v_amax[at + 1]));
      last_hh = c0.hh;
    }
    const unsigned char* stage = smem + (i % 3) * kStage;
    const bool full = a.N - c0.blk * kBlock >= kBlock;
    if constexpr (STAGE == kVStats) {
      if (full) v_stats_item<D, true>(a, stage, red, a.bh0 + c0.hh, c0.blk);
      else v_stats_item<D, false>(a, stage, red, a.bh0 + c0.hh, c0.blk);
    } else {
      if (full) v_item<D, STAGE, true>(a, stage, red, a.bh0 + c0.hh, c0.blk, mu, am);
      else v_item<D, STAGE, false>(a, stage, red, a.bh0 + c0.hh, c0.blk, mu, am);
    }
    mu = mu_next;
    c0 = c1; c1 = c2;
    advance(c2, step, a.nb, nh);
    advance(c4, step, a.nb, nh);
  }
}

// Launch 2: per-head finalization: K channel mean, V scale, g_Q.
template <int D, int BITS>
__global__ void prep_finalize_kernel(const PrepArgs a, int which) {
  // which 0 / 2: a block of 8 D threads per head; the block partial sums are added in double, in
  // eight interleaved slices that are then added in a fixed order
  __shared__ double part[8][D];
  const int bh = a.bh0 + blockIdx.x, c = threadIdx.x % D, slice = threadIdx.x / D;
  if (which == 0 || which == 2) {
    if (which == 0 && (a.flags & VC_FLAG_K_SMOOTH)) {
      double s = 0.0;
      for (int j = slice; j < a.nb; j += 8) s += (double)a.k_part[((size_t)bh * a.nb + j) * D + c];
      part[slice][c] = s;
      __syncthreads();
    }
    if (slice == 0) {
      if (which == 2) {        // statistics from the caller: the mean as given (zero if K smoothing is off)
        a.k_mean[(size_t)bh * D + c] = (a.flags & VC_FLAG_K_SMOOTH) ? a.ext_k_mean[(size_t)bh * D + c] : 0.f;
      } else {
        double s = 0.0;
        if (a.flags & VC_FLAG_K_SMOOTH)
          for (int k = 0; k < 8; ++k) s += part[k][c];
        a.k_mean[(size_t)bh * D + c] = (float)(s / (double)a.N);
      }
      float vs = 1.0f;
      if (BITS == 8) {
        const float am = __uint_as_float(a.v_amax[(size_t)bh * D + c]);
        vs = am > 0.f ? am / 448.0f : 1.0f;
      }
      a.v_scale[(size_t)bh * D + c] = vs;
    }
    if (BITS == 4 && threadIdx.x == 0) {
      const float am = __uint_as_float(a.qk_amax[bh]);
      a.q_scale[bh] = am > 0.f ? am / 2688.0f : 1.0f;
    }
  } else if (BITS == 4 && threadIdx.x == 0) {
    const float am = __uint_as_float(a.qk_amax[a.BH + bh]);
    a.k_scale[bh] = am > 0.f ? am / 2688.0f : 1.0f;
  }
}

// Q/K pass: STAGE = amax (4-bit head amax of tensor z0), or quantization of Q (z = 0) and K
// (z = 1).  A warp owns 32 / TPR rows of the block from end to end: it copies them in (consecutive
// lanes on consecutive 16-byte chunks, the source rows taken from a small ring of permutation
// entries in shared memory), its threads read their rows from the padded tile, and the rows'
// codes leave through the warp's slice of a swizzled tile, again with full-line stores.  So the
// data needs warp-level synchronization only; the one CTA-wide barrier per item is the exchange
// of the block maximum.
// Shared memory: [2 stages x 128 x pitch][out tile 128 x D][src ring 3 x 128][scratch][RoPE table].
// FAST: the packed row transform (standard configuration), see qk_row_item_fast.
template <int D, int STAGE, int TPR, bool FAST = false>
__global__ void __launch_bounds__(kRowThreads * TPR, 2) prep_qk_kernel(const PrepArgs a, int n_items, int nh, int z0) {
  constexpr int NT = kRowThreads * TPR;
  constexpr int kRowBytes = STAGE == kStageQuant4 ? D / 2 : D;      // code bytes per row
  constexpr int CPR = kRowBytes / 16;                                // 16-byte chunks per code row
  constexpr int RW = 32 / TPR;                                       // rows of a warp
  constexpr int LPR = D / 8;                                         // lanes on one input row
  constexpr int RPI = 32 / LPR;                                      // input rows per warp instruction
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char* out_tile = smem + 2 * Geo<D>::stage_bytes;
  int* src_ring = reinterpret_cast<int*>(out_tile + kBlock * D);     // [3][128]
  float* red = reinterpret_cast<float*>(src_ring + 3 * kBlock);      // [2][16]
  float* kmean_s = red + 32;                                         // [D]
  const int tid = threadIdx.x, lane = tid & 31, row0 = (tid >> 5) * RW;
  if (FAST) {
    for (int c = tid; c < D; c += NT) kmean_s[c] = 0.f;    // (m+, m-) pairs: zeros until a smoothed K head arrives
  }
  const RopeTab tab = stage_rope_table(a, reinterpret_cast<unsigned char*>(kmean_s + D), FAST);
  const int my_row = qk_row_of<TPR>(tid);
  const CursorStep step = cursor_step(a.nb);
  auto fetch = [&](int item, const Cursor& c) -> int {   // input row behind row `row0 + lane` of the item, -1 if none
    if (item >= n_items || lane >= RW) return -1;
    const int t = c.blk * kBlock + row0 + lane;
    if (t >= a.N) return -1;
    // the head amax is a maximum over all rows: that stage reads the rows in place
    const bool gather = (c.z + z0) == 1 && a.perm != nullptr && STAGE != kStageAmax;
    return gather ? min(max(__ldg(&a.perm[(size_t)(a.bh0 + c.hh) * a.N + t]), 0), a.N - 1) : t;   // clamped: never a bad address
  };
  auto issue = [&](int item, const Cursor& c, int st, const int* src) {
    if (item < n_items) {
      const char* base = reinterpret_cast<const char*>((c.z + z0) == 0 ? a.q : a.k) + head_offset_bytes(a, a.bh0 + c.hh) + 16 * (lane % LPR);
      unsigned char* dst = smem + st * Geo<D>::stage_bytes + 16 * (lane % LPR) + (row0 + lane / LPR) * Geo<D>::pitch;
#pragma unroll
      for (int k = 0; k < RW / RPI; ++k) {
        const int sr = src[row0 + lane / LPR + k * RPI];
        if (sr >= 0) cp_async16(dst + k * RPI * Geo<D>::pitch, base + (int64_t)sr * a.stride_n_bytes);
      }
    }
    cp_async_commit();
  };
  // cursors of items i, i+1 and i+3 of this CTA
  const int g = gridDim.x;
  Cursor c0 = cursor_at(blockIdx.x, a.nb, nh), c1 = c0;
  advance(c1, step, a.nb, nh);
  Cursor c3 = c1;
  advance(c3, step, a.nb, nh);
  if (lane < RW) {
    src_ring[row0 + lane] = fetch(blockIdx.x, c0);
    src_ring[kBlock + row0 + lane] = fetch(blockIdx.x + g, c1);
  }
  int nxt = fetch(blockIdx.x + 2 * g, c3);    // (c3 still stands at item 2 here)
  advance(c3, step, a.nb, nh);
  __syncwarp();
  issue(blockIdx.x, c0, 0, src_ring);
  int i = 0, last_hh = -1;
  for (int item = blockIdx.x; item < n_items; item += g, ++i) {
    cp_async_wait<0>();                       // my chunks of item i have landed ...
    __syncwarp();                             // ... and the warp's; the warp is done with item i-1
    if (lane < RW) src_ring[((i + 2) % 3) * kBlock + row0 + lane] = nxt;
    nxt = fetch(item + 3 * g, c3);
    issue(item + g, c1, (i + 1) & 1, src_ring + ((i + 1) % 3) * kBlock);
    const unsigned char* stage = smem + (i & 1) * Geo<D>::stage_bytes;
    const int s0 = src_ring[(i % 3) * kBlock + my_row];
    const int tensor = c0.z + z0, bh = a.bh0 + c0.hh;
    if constexpr (FAST)
      qk_row_item_fast<D, STAGE, TPR>(a, tensor, stage, out_tile, red, kmean_s, tab.saddr, bh, c0.blk, i, tensor == 1 && c0.hh != last_hh, s0);
    else
      qk_row_item<D, STAGE, TPR>(a, tensor, stage, out_tile, red, kmean_s, tab, bh, c0.blk, i, tensor == 1 && c0.hh != last_hh, s0);
    if (tensor == 1) last_hh = c0.hh;
    if constexpr (STAGE != kStageAmax) {
      __syncwarp();                           // the warp's rows of the code tile are complete
      uint4* gdst = reinterpret_cast<uint4*>((tensor == 0 ? a.q_codes : a.k_codes) + ((size_t)bh * a.n_pad + (size_t)c0.blk * kBlock + row0) * kRowBytes) + lane;
#pragma unroll
      for (int k = 0; k < CPR * RW / 32; ++k) {
        const int idx = k * 32 + lane, row = row0 + idx / CPR, chunk = idx % CPR;
        const int sw = (row / (8 / CPR)) & (CPR - 1);
        gdst[k * 32] = *reinterpret_cast<const uint4*>(out_tile + row * kRowBytes + ((chunk ^ sw) << 4));
      }
    }
    c0 = c1;
    advance(c1, step, a.nb, nh);
    advance(c3, step, a.nb, nh);
  }
}

template <typename K>
cudaError_t allow_smem(K kernel, size_t bytes) {
  return bytes > 48 * 1024 ? cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) : cudaSuccess;
}

int persistent_grid(int n_items, int per_sm = 2) {
  // SM count of the CURRENT device (cached per device: a process may drive GPUs of different sizes)
  static int cache[64] = {};
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) dev = -1;
  if (dev >= 0 && dev < 64 && cache[dev] > 0) sms = cache[dev];
  else {
    if (dev < 0 || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) sms = 148;
    if (dev >= 0 && dev < 64) cache[dev] = sms;
  }
  const int g = per_sm * sms;
  return n_items < g ? n_items : g;
}

template <int D, int BITS>
cudaError_t run(const Problem& pr, PrepArgs a, const WorkLayout& wl, uint8_t* work, cudaStream_t s) {
  const size_t rope_bytes = ((a.flags & VC_FLAG_ROPE) && a.rope_in_smem) ? (size_t)a.rd.entries * 8 : 0;
  const size_t colsum_smem = 2 * (size_t)kThreads * (D / 16) * 16 + 8 * D * 4 + rope_bytes;
  const size_t row_smem = 2 * (size_t)Geo<D>::stage_bytes + (size_t)kBlock * D + 3 * kBlock * 4 + 128 + D * 4 + rope_bytes;
  const size_t v_smem = 3 * (size_t)kBlock * 2 * D + 16 * D * 4 + 2 * kBlock * 4;
  constexpr int kQuant = BITS == 8 ? kStageQuant8 : kStageQuant4;
  constexpr int kTpr = VC_PREP_TPR;            // threads per Q/K row
  constexpr int kTprF = D == 128 ? VC_PREP_TPR_FAST : VC_PREP_TPR;   // ... of the packed row transform
  constexpr int kVQuant = BITS == 8 ? kVQuant8 : kVQuant4;
  cudaError_t e;
  if ((e = allow_smem(prep_kcolsum_kernel<D>, colsum_smem)) != cudaSuccess) return e;
  if ((e = allow_smem(prep_v_kernel<D, kVStats>, v_smem)) != cudaSuccess) return e;
  if ((e = allow_smem(prep_v_kernel<D, kVQuant>, v_smem)) != cudaSuccess) return e;
  if (BITS == 4 && (e = allow_smem(prep_v_kernel<D, kVQuant4M>, v_smem)) != cudaSuccess) return e;
  const bool v_pow2 = hybrid4(pr);           // 4-bit values under power-of-two factors per 32 tokens
  if ((e = allow_smem(prep_qk_kernel<D, kQuant, kTpr>, row_smem)) != cudaSuccess) return e;
  if (BITS == 8 && (e = allow_smem(prep_qk_kernel<D, kStageQuant8I, kTpr>, row_smem)) != cudaSuccess) return e;
  if (BITS == 8 && (e = allow_smem(prep_qk_kernel<D, kStageQuant8, kTprF, true>, row_smem)) != cudaSuccess) return e;
  if (BITS == 8 && (e = allow_smem(prep_qk_kernel<D, kStageQuant8I, kTprF, true>, row_smem)) != cudaSuccess) return e;
  // the packed row transform serves the standard configuration
  const bool fast = (a.flags & VC_FLAG_ROPE) && (a.flags & VC_FLAG_HADAMARD) && a.rope_default && a.rope_in_smem;
  if (BITS == 4 && (e = allow_smem(prep_qk_kernel<D, kStageAmax, kTpr>, row_smem)) != cudaSuccess) return e;
  if (BITS == 4 && (e = allow_smem(prep_qk_kernel<D, kStageAmax, kTprF, true>, row_smem)) != cudaSuccess) return e;
  if (BITS == 4 && (e = allow_smem(prep_qk_kernel<D, kStageQuant4, kTprF, true>, row_smem)) != cudaSuccess) return e;
  int group = pr.heads_per_pass > 0 ? pr.heads_per_pass : pr.BH;
  if (group > 32768) group = 32768;
  for (int bh0 = 0; bh0 < pr.BH; bh0 += group) {
    const int nh = pr.BH - bh0 < group ? pr.BH - bh0 : group;
    const int per = pr.nb * nh;
    a.bh0 = bh0;
    const bool ext = a.ext_k_mean != nullptr;     // the caller supplied the statistics: no statistics launches
    if ((a.flags & VC_FLAG_K_SMOOTH) && !ext) {
      prep_kcolsum_kernel<D><<<persistent_grid(per), kThreads, colsum_smem, s>>>(a, per, nh);
      count_launches(1);
    }
    if (BITS == 8 && !ext) { prep_v_kernel<D, kVStats><<<persistent_grid(per), kThreads, v_smem, s>>>(a, per, nh); count_launches(1); }
    auto amax_pass = [&](int z0) {
      if (fast) prep_qk_kernel<D, kStageAmax, kTprF, true><<<persistent_grid(per), kRowThreads * kTprF, row_smem, s>>>(a, per, nh, z0);
      else prep_qk_kernel<D, kStageAmax, kTpr><<<persistent_grid(per), kRowThreads * kTpr, row_smem, s>>>(a, per, nh, z0);
      count_launches(1);
    };
    if (BITS == 4) amax_pass(0);
    prep_finalize_kernel<D, BITS><<<nh, 8 * D, 0, s>>>(a, ext ? 2 : 0);
    count_launches(1);
    if (BITS == 4) {
      amax_pass(1);
      prep_finalize_kernel<D, BITS><<<nh, 32, 0, s>>>(a, 1);
      count_launches(1);
    }
    if constexpr (BITS == 8) {
      if (fast && (a.flags & VC_FLAG_INT8_QK))
        prep_qk_kernel<D, kStageQuant8I, kTprF, true><<<persistent_grid(2 * per), kRowThreads * kTprF, row_smem, s>>>(a, 2 * per, nh, 0);
      else if (fast)
        prep_qk_kernel<D, kStageQuant8, kTprF, true><<<persistent_grid(2 * per), kRowThreads * kTprF, row_smem, s>>>(a, 2 * per, nh, 0);
      else if (a.flags & VC_FLAG_INT8_QK)
        prep_qk_kernel<D, kStageQuant8I, kTpr><<<persistent_grid(2 * per), kRowThreads * kTpr, row_smem, s>>>(a, 2 * per, nh, 0);
      else
        prep_qk_kernel<D, kStageQuant8, kTpr><<<persistent_grid(2 * per), kRowThreads * kTpr, row_smem, s>>>(a, 2 * per, nh, 0);
    } else {
      if (fast) prep_qk_kernel<D, kStageQuant4, kTprF, true><<<persistent_grid(2 * per), kRowThreads * kTprF, row_smem, s>>>(a, 2 * per, nh, 0);
      else prep_qk_kernel<D, kStageQuant4, kTpr><<<persistent_grid(2 * per), kRowThreads * kTpr, row_smem, s>>>(a, 2 * per, nh, 0);
    }
    if (BITS == 4 && v_pow2)
      prep_v_kernel<D, kVQuant4M><<<persistent_grid(per), kThreads, v_smem, s>>>(a, per, nh);
    else
      prep_v_kernel<D, kVQuant><<<persistent_grid(per), kThreads, v_smem, s>>>(a, per, nh);
    count_launches(2);
  }
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_prep(const Problem& pr, const QuantLayout& ql, const WorkLayout& wl,
                        const void* q, const void* k, const void* v, const int32_t* perm,
                        uint8_t* quant, uint8_t* work, cudaStream_t stream, const vc_prep_stats* stats) {
  PrepArgs a{};
  a.q = (const __nv_bfloat16*)q; a.k = (const __nv_bfloat16*)k; a.v = (const __nv_bfloat16*)v;
  a.perm = perm;
  a.stride_b = pr.stride_b; a.stride_h = pr.stride_h; a.stride_n = pr.stride_n;
  a.stride_n_bytes = (int)(2 * pr.stride_n);
  a.mul_H = ((1ull << 40) + pr.H - 1) / pr.H;
  a.H = pr.H; a.N = pr.N; a.n_pad = pr.n_pad; a.nb = pr.nb; a.bh0 = 0; a.flags = pr.flags; a.BH = pr.BH;
  a.q_codes = quant + ql.q_codes; a.k_codes = quant + ql.k_codes; a.v_codes = quant + ql.v_codes;
  a.q_micro = quant + ql.q_micro; a.k_micro = quant + ql.k_micro; a.v_micro = quant + ql.v_micro;
  a.q_scale = (float*)(quant + ql.q_scale); a.k_scale = (float*)(quant + ql.k_scale);
  a.v_scale = (float*)(quant + ql.v_scale); a.k_mean = (float*)(quant + ql.k_mean);
  a.v_means = (__nv_bfloat16*)(quant + ql.v_means);
  a.rope = (const float2*)(work + wl.rope);
  a.k_part = (float*)(work + wl.k_part); a.v_mu = (float*)(work + wl.v_mu);
  a.v_amax = (unsigned int*)(work + wl.amax);
  a.qk_amax = a.v_amax + (size_t)pr.BH * pr.d;
  const bool ext = stats != nullptr;
  if (ext) {   // K mean, V block means and residual maxima as the caller computed them
    a.ext_k_mean = stats->k_mean;
    a.v_mu = const_cast<float*>(stats->v_block_mean);
    a.v_amax = reinterpret_cast<unsigned int*>(const_cast<float*>(stats->v_amax));
  }
  const int len[3] = {pr.grid_t, pr.grid_h, pr.grid_w};
  int ps = 0;
  for (int ax = 0; ax < 3; ++ax) {
    a.rd.pair_start[ax] = ps;
    a.rd.pairs[ax] = pr.rope_dim[ax] / 2;
    a.rd.off[ax] = wl.rope_off[ax];
    a.rd.len[ax] = len[ax];
    ps += pr.rope_dim[ax] / 2;
  }
  a.rd.entries = wl.rope_entries;
  a.rd.grid_h = pr.grid_h; a.rd.grid_w = pr.grid_w;
  a.rd.mul_w = ((1ull << 40) + pr.grid_w - 1) / pr.grid_w;
  a.rd.mul_h = ((1ull << 40) + pr.grid_h - 1) / pr.grid_h;
  a.rope_in_smem = (size_t)wl.rope_entries * 8 <= 96 * 1024;
  {
    const int sdef = 2 * (pr.d / 6);
    a.rope_default = pr.rope_dim[0] == pr.d - 2 * sdef && pr.rope_dim[1] == sdef && pr.rope_dim[2] == sdef;
  }
  cudaError_t e;
  if ((e = cudaMemsetAsync(work + wl.status, 0, 4, stream)) != cudaSuccess) return e;
  if (!ext && (e = cudaMemsetAsync(work + wl.amax, 0, wl.amax_bytes, stream)) != cudaSuccess) return e;
  if (a.flags & VC_FLAG_ROPE) {
    rope_table_kernel<<<(a.rd.entries + 255) / 256, 256, 0, stream>>>(
        reinterpret_cast<float2*>(work + wl.rope), a.rd, (double)pr.rope_theta);
    count_launches(1);
  }
  if ((e = launch_perm_check(pr, perm, wl, work, stream)) != cudaSuccess) return e;
  if (pr.d == 128) return pr.bits == 8 ? run<128, 8>(pr, a, wl, work, stream) : run<128, 4>(pr, a, wl, work, stream);
  return pr.bits == 8 ? run<64, 8>(pr, a, wl, work, stream) : run<64, 4>(pr, a, wl, work, stream);
}

}  // namespace vc

// ---------------------------------------------------------------------------------------
// vc_prep_noalloc: the preprocessing pass for callers that cannot provide a workspace.
// The scratch that vc_prep takes from the caller (RoPE tables, per-block partial sums, block
// means, amax words) lives here in a fixed array in device global memory, so the call needs no
// allocation of any kind; the price is a size limit and one array per GPU for the life of the
// process.
namespace {

// Held by every GPU that loads this library until the process exits.
static __device__ __align__(256) unsigned char g_prep_scratch[VC_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
unsigned char* g_scratch_addr[kMaxDevices] = {};   // device address of the array, per device

// In host code the array's name is only a handle; the device address has to be asked for,
// once per device, with that device current.
cudaError_t scratch_address(unsigned char** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  unsigned char* ptr = __atomic_load_n(&g_scratch_addr[dev], __ATOMIC_ACQUIRE);
  if (!ptr) {
    e = cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_prep_scratch);
    if (e != cudaSuccess) return e;
    __atomic_store_n(&g_scratch_addr[dev], ptr, __ATOMIC_RELEASE);   // same value from any thread
  }
  *out = ptr;
  return cudaSuccess;
}

}  // namespace

extern "C" vc_status vc_prep_noalloc(const vc_params* p, const void* q, const void* k, const void* v,
                                     const int32_t* perm, void* quant, void* stream) {
  vc::Problem pr;
  vc_status st = vc::resolve(p, &pr);
  if (st != VC_OK) return st;
  if (!q || !k || !v || !quant) return VC_ERR_INVALID_ARG;
  if (((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)quant | (uintptr_t)perm) & 15) return VC_ERR_INVALID_ARG;
  const vc::QuantLayout ql = vc::quant_layout(pr);
  const vc::WorkLayout wl = vc::work_layout(pr);
  // the pass uses the workspace sections in front of the attention kernel's mean table
  if (wl.mu_mma > (size_t)VC_NOALLOC_SCRATCH_BYTES) return VC_ERR_SCRATCH_LIMIT;
  unsigned char* scratch = nullptr;
  if (scratch_address(&scratch) != cudaSuccess) return VC_ERR_CUDA;
  // launch_prep clears the words that must start at zero (status, amax) on the stream itself
  cudaError_t e = vc::launch_prep(pr, ql, wl, q, k, v, perm, (uint8_t*)quant, scratch, (cudaStream_t)stream, nullptr);
  return e == cudaSuccess ? VC_OK : VC_ERR_CUDA;
}
