// C-ABI entry points of libvc: argument validation, buffer layouts, launch sequencing.
#include <atomic>
#include <mutex>
#include <vector>
#include <cstring>

#include "vc_internal.h"

namespace vc {

static std::atomic<uint64_t> g_launches{0};
void count_launches(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

static std::atomic<uint32_t> g_wait_limit{0};
uint32_t wait_limit_override() { return g_wait_limit.load(std::memory_order_relaxed); }

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

vc_status resolve(const vc_params* p, Problem* out) {
  if (!p || !out) return VC_ERR_INVALID_ARG;
  Problem pr{};
  pr.B = p->B; pr.H = p->H; pr.N = p->N; pr.d = p->d;
  if (pr.B < 1 || pr.H < 1 || pr.N < 1) return VC_ERR_INVALID_ARG;
  // B * H is the second grid dimension of several launches (limit 65535)
  if ((int64_t)pr.B * pr.H > 65535 || pr.N > (1 << 22)) return VC_ERR_INVALID_ARG;
  if (pr.d != 64 && pr.d != 128) return VC_ERR_INVALID_ARG;
  pr.BH = pr.B * pr.H;
  pr.grid_t = p->grid_t; pr.grid_h = p->grid_h; pr.grid_w = p->grid_w;
  if (pr.grid_t < 1 || pr.grid_h < 1 || pr.grid_w < 1) return VC_ERR_INVALID_ARG;
  if (pr.grid_h > (1 << 18) || pr.grid_w > (1 << 18)) return VC_ERR_INVALID_ARG;
  if ((int64_t)pr.grid_t * pr.grid_h * pr.grid_w != pr.N) return VC_ERR_INVALID_ARG;
  pr.bits = p->bits;
  if (pr.bits != 8 && pr.bits != 4) return VC_ERR_INVALID_ARG;
  pr.p_format = p->p_format;
  if (pr.p_format == VC_P_DEFAULT) pr.p_format = pr.bits == 8 ? VC_P_EXPCAST_E4M3 : VC_P_NVFP4;
  if (pr.p_format < VC_P_EXPCAST_E4M3 || pr.p_format > VC_P_EXP_MIX_E4M3) return VC_ERR_INVALID_ARG;
  if (pr.bits == 8 && pr.p_format == VC_P_NVFP4) return VC_ERR_UNSUPPORTED;
  if (pr.p_format > VC_P_NVFP4 && (p->flags & VC_FLAG_INT8_QK)) return VC_ERR_UNSUPPORTED;
  if (pr.bits == 4 && pr.p_format != VC_P_NVFP4 && pr.p_format != VC_P_EXPCAST_E4M3) return VC_ERR_UNSUPPORTED;
  pr.flags = p->flags;
  if (pr.flags & ~(VC_FLAG_ALL | VC_FLAG_INT8_QK | VC_FLAG_CHECK_PERM)) return VC_ERR_INVALID_ARG;
  // scale blocks and the value block of Eq. 4: the kernels implement 128 only
  if (p->block_q < 0 || p->block_k < 0 || p->block_v < 0) return VC_ERR_INVALID_ARG;
  if ((p->block_q && p->block_q != kBlock) || (p->block_k && p->block_k != kBlock) || (p->block_v && p->block_v != kBlock))
    return VC_ERR_UNSUPPORTED;
  pr.softmax_scale = p->softmax_scale != 0.f ? p->softmax_scale : 1.0f / sqrtf((float)pr.d);
  if (!(pr.softmax_scale > 0.f)) return VC_ERR_INVALID_ARG;
  pr.beta = p->beta != 0.f ? p->beta : -0.35f;
  pr.rope_theta = p->rope_theta != 0.f ? p->rope_theta : 10000.0f;
  if (p->rope_dim_t == 0 && p->rope_dim_h == 0 && p->rope_dim_w == 0) {
    int s = 2 * (pr.d / 6);
    pr.rope_dim[0] = pr.d - 2 * s; pr.rope_dim[1] = s; pr.rope_dim[2] = s;
  } else {
    pr.rope_dim[0] = p->rope_dim_t; pr.rope_dim[1] = p->rope_dim_h; pr.rope_dim[2] = p->rope_dim_w;
  }
  int sum = 0;
  for (int a = 0; a < 3; ++a) {
    if (pr.rope_dim[a] < 0 || (pr.rope_dim[a] & 1)) return VC_ERR_INVALID_ARG;
    sum += pr.rope_dim[a];
  }
  if (sum != pr.d) return VC_ERR_INVALID_ARG;
  pr.stride_n = p->stride_n ? p->stride_n : pr.d;
  pr.stride_h = p->stride_h ? p->stride_h : (int64_t)pr.N * pr.d;
  pr.stride_b = p->stride_b ? p->stride_b : (int64_t)pr.H * pr.N * pr.d;
  if (pr.stride_n >= (1ll << 30)) return VC_ERR_UNSUPPORTED;     // a row stride in bytes fits 32 bits
  if (pr.stride_n < pr.d || (pr.stride_n % 8) || (pr.stride_h % 8) || (pr.stride_b % 8))
    return VC_ERR_INVALID_ARG;   // rows are read with 16-byte vector loads
  pr.n_pad = kBlock * ((pr.N + kBlock - 1) / kBlock);
  pr.nb = pr.n_pad / kBlock;
  pr.heads_per_pass = p->heads_per_pass > 0 ? p->heads_per_pass : 0;
  pr.kernel_variant = p->kernel_variant;
  if (pr.kernel_variant < 0 || pr.kernel_variant > 1) return VC_ERR_INVALID_ARG;
  if ((pr.flags & VC_FLAG_INT8_QK) && (pr.bits != 8 || pr.kernel_variant != 0)) return VC_ERR_INVALID_ARG;
  if (hybrid4(pr) && pr.kernel_variant != 0) return VC_ERR_UNSUPPORTED;
  *out = pr;
  return VC_OK;
}

QuantLayout quant_layout(const Problem& pr) {
  QuantLayout L{};
  const size_t BH = pr.BH, np_ = pr.n_pad, d = pr.d, nb = pr.nb;
  const bool four = pr.bits == 4;
  L.q_codes_bytes = four ? BH * np_ * d / 2 : BH * np_ * d;
  L.k_codes_bytes = L.q_codes_bytes;
  L.v_codes_bytes = L.q_codes_bytes;
  L.q_scale_bytes = four ? BH * 4 : BH * nb * 4;
  L.k_scale_bytes = L.q_scale_bytes;
  L.v_scale_bytes = BH * d * 4;
  L.v_means_bytes = BH * nb * d * 2;
  L.k_mean_bytes = BH * d * 4;
  L.q_micro_bytes = four ? BH * np_ * d / 16 : 0;
  L.k_micro_bytes = L.q_micro_bytes;
  L.v_micro_bytes = hybrid4(pr) ? BH * np_ * d / 32 : L.q_micro_bytes;
  size_t off = 0;
  auto place = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 1024); return o; };
  L.q_codes = place(L.q_codes_bytes);
  L.k_codes = place(L.k_codes_bytes);
  L.v_codes = place(L.v_codes_bytes);
  L.q_scale = place(L.q_scale_bytes);
  L.k_scale = place(L.k_scale_bytes);
  L.v_scale = place(L.v_scale_bytes);
  L.v_means = place(L.v_means_bytes);
  L.k_mean = place(L.k_mean_bytes);
  L.q_micro = place(L.q_micro_bytes);
  L.k_micro = place(L.k_micro_bytes);
  L.v_micro = place(L.v_micro_bytes);
  L.total = off;
  return L;
}

WorkLayout work_layout(const Problem& pr) {
  WorkLayout W{};
  const size_t BH = pr.BH, d = pr.d, nb = pr.nb;
  const int len[3] = {pr.grid_t, pr.grid_h, pr.grid_w};
  int e = 0;
  for (int a = 0; a < 3; ++a) { W.rope_off[a] = e; e += len[a] * (pr.rope_dim[a] / 2); }
  W.rope_entries = e;
  size_t off = 0;
  auto place = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 1024); return o; };
  W.status = place(256);
  W.rope = place((size_t)e * 16);   // (cos, sin) entries, then the same entries as (cos + sin, cos - sin)
  W.k_part = place(BH * nb * d * 4);
  W.v_mu = place(BH * nb * d * 4);
  W.amax_bytes = BH * d * 4 + 2 * BH * 4;
  W.amax = place(W.amax_bytes);
  W.perm_bits_bytes = (pr.flags & VC_FLAG_CHECK_PERM) ? BH * (((size_t)pr.N + 31) / 32) * 4 : 0;
  W.perm_bits = place(W.perm_bits_bytes);
  W.mu_mma = place(BH * nb * d * 32);
  W.sf_q = place(pr.bits == 4 ? BH * nb * (d / 64) * 512 : 0);
  W.sf_kv = place(pr.bits == 4 ? BH * nb * (d / 64 + 2) * 512 : 0);
  W.expand = place(pr.bits == 4 && pr.kernel_variant == 1 ? 3 * BH * (size_t)pr.n_pad * d * 2 : 0);
  W.total = off;
  return W;
}

static bool misaligned(const void* p) { return ((uintptr_t)p & 15) != 0; }

// Helper streams and events of vc_attn_host, one set per device.
constexpr int kMaxHostPipes = 64;
struct HostPipe {
  std::mutex mu;
  cudaStream_t s_in = nullptr, s_out = nullptr;
  std::vector<cudaEvent_t> ev;
};
static HostPipe g_host_pipes[kMaxHostPipes];

}  // namespace vc

using namespace vc;

extern "C" {

size_t vc_quant_bytes(const vc_params* p) {
  Problem pr;
  if (resolve(p, &pr) != VC_OK) return 0;
  return quant_layout(pr).total;
}

size_t vc_workspace_bytes(const vc_params* p) {
  Problem pr;
  if (resolve(p, &pr) != VC_OK) return 0;
  return work_layout(pr).total;
}

static vc_status prep_impl(const vc_params* p, const void* q, const void* k, const void* v, const int32_t* perm,
                           const vc_prep_stats* stats, void* quant, void* workspace, void* stream) {
  Problem pr;
  vc_status st = resolve(p, &pr);
  if (st != VC_OK) return st;
  if (!q || !k || !v || !quant || !workspace) return VC_ERR_INVALID_ARG;
  if (misaligned(q) || misaligned(k) || misaligned(v) || misaligned(quant) ||
      misaligned(workspace) || (perm && misaligned(perm)))
    return VC_ERR_INVALID_ARG;
  QuantLayout ql = quant_layout(pr);
  WorkLayout wl = work_layout(pr);
  if (stats) {
    if (pr.bits != 8) return VC_ERR_UNSUPPORTED;   // at 4 bits the outer scales of Q and K are statistics too
    if (!stats->k_mean || !stats->v_block_mean || !stats->v_amax) return VC_ERR_INVALID_ARG;
    if (misaligned(stats->k_mean) || misaligned(stats->v_block_mean) || misaligned(stats->v_amax)) return VC_ERR_INVALID_ARG;
  }
  cudaError_t e = launch_prep(pr, ql, wl, q, k, v, perm, (uint8_t*)quant, (uint8_t*)workspace,
                              (cudaStream_t)stream, stats);
  return e == cudaSuccess ? VC_OK : VC_ERR_CUDA;
}

vc_status vc_prep(const vc_params* p, const void* q, const void* k, const void* v,
                  const int32_t* perm, void* quant, void* workspace, void* stream) {
  return prep_impl(p, q, k, v, perm, nullptr, quant, workspace, stream);
}

vc_status vc_prep_with_stats(const vc_params* p, const void* q, const void* k, const void* v, const int32_t* perm,
                             const vc_prep_stats* stats, void* quant, void* workspace, void* stream) {
  if (!stats) return VC_ERR_INVALID_ARG;
  return prep_impl(p, q, k, v, perm, stats, quant, workspace, stream);
}

vc_status vc_prep_stats_view(const vc_params* p, const void* quant, const void* workspace, vc_prep_stats* out) {
  Problem pr;
  vc_status st = resolve(p, &pr);
  if (st != VC_OK) return st;
  if (!quant || !workspace || !out) return VC_ERR_INVALID_ARG;
  if (pr.bits != 8) return VC_ERR_UNSUPPORTED;
  const QuantLayout ql = quant_layout(pr);
  const WorkLayout wl = work_layout(pr);
  out->k_mean = (const float*)((const uint8_t*)quant + ql.k_mean);
  out->v_block_mean = (const float*)((const uint8_t*)workspace + wl.v_mu);
  out->v_amax = (const float*)((const uint8_t*)workspace + wl.amax);
  return VC_OK;
}

static vc_status attn_fwd_impl(const vc_params* p, const void* quant, void* o, void* workspace, void* stream, bool clear_status) {
  Problem pr;
  vc_status st = resolve(p, &pr);
  if (st != VC_OK) return st;
  if (!quant || !o || !workspace) return VC_ERR_INVALID_ARG;
  if (misaligned(quant) || misaligned(o) || misaligned(workspace)) return VC_ERR_INVALID_ARG;
  // the 4-bit tensor map of the hybrid arrangement's value codes wants a 32-byte aligned base
  if (hybrid4(pr) && ((uintptr_t)quant & 31)) return VC_ERR_INVALID_ARG;
  QuantLayout ql = quant_layout(pr);
  WorkLayout wl = work_layout(pr);
  cudaError_t e = launch_attn_fwd(pr, ql, wl, (const uint8_t*)quant, o, (uint8_t*)workspace,
                                  (cudaStream_t)stream, clear_status);
  if (e == cudaErrorNotSupported) return VC_ERR_UNSUPPORTED;
  return e == cudaSuccess ? VC_OK : VC_ERR_CUDA;
}

vc_status vc_attn_fwd(const vc_params* p, const void* quant, void* o, void* workspace, void* stream) {
  return attn_fwd_impl(p, quant, o, workspace, stream, true);
}

vc_status vc_attn(const vc_params* p, const void* q, const void* k, const void* v,
                  const int32_t* perm, void* o, void* quant, void* workspace, void* stream) {
  vc_status st = vc_prep(p, q, k, v, perm, quant, workspace, stream);
  if (st != VC_OK) return st;
  return attn_fwd_impl(p, quant, o, workspace, stream, false);   // keeps what the pass recorded in the status word
}

vc_status vc_attn_host(const vc_params* p, const void* q_host, const void* k_host,
                       const void* v_host, const int32_t* perm_host, void* o_host,
                       void* q_dev, void* k_dev, void* v_dev, int32_t* perm_dev, void* o_dev,
                       void* quant, void* workspace, void* stream) {
  Problem pr;
  vc_status st = resolve(p, &pr);
  if (st != VC_OK) return st;
  if (!q_host || !k_host || !v_host || !o_host || !q_dev || !k_dev || !v_dev || !o_dev)
    return VC_ERR_INVALID_ARG;
  if (perm_host && !perm_dev) return VC_ERR_INVALID_ARG;
  if (p->stride_b || p->stride_h || p->stride_n) {
    if (pr.stride_n != pr.d || pr.stride_h != (int64_t)pr.N * pr.d ||
        pr.stride_b != (int64_t)pr.H * pr.N * pr.d)
      return VC_ERR_INVALID_ARG;   // host buffers are packed
  }
  // Heads are independent, so the call is pipelined over groups of heads: while group g is
  // computed on `stream`, group g+1 is on its way in on a copy stream and group g-1 on its
  // way out on another (PCIe is full duplex).  The bundle and workspace are reused by every
  // group, which is safe because the groups' kernels run in order on `stream`.
  cudaStream_t s = (cudaStream_t)stream;
  // heads per group: about a tenth of the heads, in multiples that keep a group's slice of
  // perm 16-byte aligned (N * 4 bytes per head).  The input copy is the longest of the three
  // pipelined activities, so what the call costs beyond it is the first group's copy (nothing
  // can run before it) and the last group's compute and output copy: the groups at both ends are
  // small (1, 2, ... and ..., 2, 1 multiples), the ones in between large enough to run efficiently.
  const int mult = pr.N % 4 == 0 ? 1 : (pr.N % 2 == 0 ? 2 : 4);
  int hg = pr.BH >= 10 ? (pr.BH + 9) / 10 : 1;
  hg = (hg + mult - 1) / mult * mult;
  std::vector<int> sizes;
  if (pr.BH >= 12 * mult && hg > 2 * mult) {
    const int last = mult + pr.BH % mult;              // the last group absorbs a remainder
    int middle = pr.BH - last - 2 * mult - 3 * mult;   // after the leading 1, 2 and before the trailing 2, 1
    sizes.push_back(mult);
    sizes.push_back(2 * mult);
    for (; middle > 0; middle -= hg) sizes.push_back(middle < hg ? middle : hg);
    sizes.push_back(2 * mult);
    sizes.push_back(last);
  } else {
    for (int h = 0; h < pr.BH; h += hg) sizes.push_back(pr.BH - h < hg ? pr.BH - h : hg);
  }
  const int groups = (int)sizes.size();
  const size_t head_elems = (size_t)pr.N * pr.d;
  // The two helper streams and the events are made once per device and kept for the life of the
  // process (a call used to create and destroy 2 streams and 2 * groups + 2 events); calls on one
  // device take turns, which costs nothing: a call ends with the stream synchronized anyway.
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxHostPipes) return VC_ERR_CUDA;
  HostPipe& hp = g_host_pipes[dev];
  std::lock_guard<std::mutex> lock(hp.mu);
  bool ok = true;
  if (!hp.s_in) ok = cudaStreamCreateWithFlags(&hp.s_in, cudaStreamNonBlocking) == cudaSuccess;
  if (ok && !hp.s_out) ok = cudaStreamCreateWithFlags(&hp.s_out, cudaStreamNonBlocking) == cudaSuccess;
  while (ok && hp.ev.size() < (size_t)(2 * groups + 2)) {
    cudaEvent_t e = nullptr;
    ok = cudaEventCreateWithFlags(&e, cudaEventDisableTiming) == cudaSuccess;
    if (ok) hp.ev.push_back(e);
  }
  cudaStream_t s_in = hp.s_in, s_out = hp.s_out;
  std::vector<cudaEvent_t>& ev = hp.ev;
  vc_status result = VC_OK;
  if (ok) {
    cudaEvent_t e_begin = ev[2 * groups], e_end = ev[2 * groups + 1];
    ok = cudaEventRecord(e_begin, s) == cudaSuccess && cudaStreamWaitEvent(s_in, e_begin, 0) == cudaSuccess &&
         cudaStreamWaitEvent(s_out, e_begin, 0) == cudaSuccess;
    vc_params sub = *p;
    sub.B = 1;
    sub.stride_b = sub.stride_h = sub.stride_n = 0;
    int h0 = 0;
    for (int g = 0; ok && g < groups; h0 += sizes[g], ++g) {
      const int nh = sizes[g];
      const size_t off = (size_t)h0 * head_elems * 2, bytes = (size_t)nh * head_elems * 2;
      ok = cudaMemcpyAsync((char*)q_dev + off, (const char*)q_host + off, bytes, cudaMemcpyHostToDevice, s_in) == cudaSuccess &&
           cudaMemcpyAsync((char*)k_dev + off, (const char*)k_host + off, bytes, cudaMemcpyHostToDevice, s_in) == cudaSuccess &&
           cudaMemcpyAsync((char*)v_dev + off, (const char*)v_host + off, bytes, cudaMemcpyHostToDevice, s_in) == cudaSuccess;
      if (ok && perm_host)
        ok = cudaMemcpyAsync(perm_dev + (size_t)h0 * pr.N, perm_host + (size_t)h0 * pr.N, (size_t)nh * pr.N * 4,
                             cudaMemcpyHostToDevice, s_in) == cudaSuccess;
      ok = ok && cudaEventRecord(ev[2 * g], s_in) == cudaSuccess && cudaStreamWaitEvent(s, ev[2 * g], 0) == cudaSuccess;
      if (!ok) break;
      sub.H = nh;
      const vc_status st_g = vc_attn(&sub, (char*)q_dev + off, (char*)k_dev + off, (char*)v_dev + off,
                                     perm_host ? perm_dev + (size_t)h0 * pr.N : nullptr, (char*)o_dev + off, quant,
                                     workspace, stream);
      if (st_g != VC_OK) { result = st_g; break; }
      ok = cudaEventRecord(ev[2 * g + 1], s) == cudaSuccess && cudaStreamWaitEvent(s_out, ev[2 * g + 1], 0) == cudaSuccess &&
           cudaMemcpyAsync((char*)o_host + off, (char*)o_dev + off, bytes, cudaMemcpyDeviceToHost, s_out) == cudaSuccess;
    }
    // join: `stream` is complete only when the last output copy is
    if (cudaEventRecord(e_end, s_out) != cudaSuccess || cudaStreamWaitEvent(s, e_end, 0) != cudaSuccess) ok = false;
    if (cudaStreamSynchronize(s_in) != cudaSuccess) ok = false;
    if (cudaStreamSynchronize(s) != cudaSuccess) ok = false;
  }
  if (cudaStreamSynchronize(s_out) != cudaSuccess) ok = false;   // the shared helpers are idle when the lock is released
  if (result != VC_OK) return result;
  return ok ? VC_OK : VC_ERR_CUDA;
}

vc_status vc_quant_view(const vc_params* p, const void* quant, vc_quant_ptrs* out) {
  Problem pr;
  vc_status st = resolve(p, &pr);
  if (st != VC_OK) return st;
  if (!quant || !out) return VC_ERR_INVALID_ARG;
  QuantLayout L = quant_layout(pr);
  uint8_t* b = (uint8_t*)quant;
  std::memset(out, 0, sizeof(*out));
  out->q_codes = b + L.q_codes; out->k_codes = b + L.k_codes; out->v_codes = b + L.v_codes;
  out->q_scale = (float*)(b + L.q_scale); out->k_scale = (float*)(b + L.k_scale);
  out->v_scale = (float*)(b + L.v_scale);
  out->v_means = b + L.v_means;
  out->k_mean = (float*)(b + L.k_mean);
  if (pr.bits == 4) {
    out->q_micro = b + L.q_micro; out->k_micro = b + L.k_micro; out->v_micro = b + L.v_micro;
  }
  out->q_codes_bytes = L.q_codes_bytes; out->k_codes_bytes = L.k_codes_bytes;
  out->v_codes_bytes = L.v_codes_bytes; out->q_scale_bytes = L.q_scale_bytes;
  out->k_scale_bytes = L.k_scale_bytes; out->v_scale_bytes = L.v_scale_bytes;
  out->v_means_bytes = L.v_means_bytes; out->k_mean_bytes = L.k_mean_bytes;
  out->q_micro_bytes = L.q_micro_bytes; out->k_micro_bytes = L.k_micro_bytes;
  out->v_micro_bytes = L.v_micro_bytes;
  return VC_OK;
}

vc_status vc_poll_status(void* workspace, void* stream) {
  if (!workspace) return VC_ERR_INVALID_ARG;
  uint32_t word = 0;
  cudaStream_t s = (cudaStream_t)stream;
  if (cudaMemcpyAsync(&word, workspace, 4, cudaMemcpyDeviceToHost, s) != cudaSuccess) return VC_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return VC_ERR_CUDA;
  if (word != 0) {
    cudaMemsetAsync(workspace, 0, 4, s);
    cudaStreamSynchronize(s);
    return (word & kStatusTimeout) ? VC_ERR_TIMEOUT : VC_ERR_INVALID_ARG;
  }
  return VC_OK;
}

int32_t vc_group_schedule(int32_t step, int32_t n_steps, int32_t reuse) {
  if (step < 0 || step >= n_steps || reuse < 1) return -1;
  const int32_t window = (n_steps + 3) / 4;          // ceil(n / 4)
  if (step >= window) return VC_GROUP_FROZEN;
  return step % reuse == 0 ? VC_GROUP_RECOMPUTE : VC_GROUP_REUSE;
}

void vc_test_set_wait_limit(uint32_t polls) { g_wait_limit.store(polls, std::memory_order_relaxed); }

uint64_t vc_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* vc_status_string(vc_status s) {
  switch (s) {
    case VC_OK: return "ok";
    case VC_ERR_INVALID_ARG: return "invalid argument";
    case VC_ERR_UNSUPPORTED: return "unsupported configuration";
    case VC_ERR_WORKSPACE: return "workspace error";
    case VC_ERR_CUDA: return "CUDA error";
    case VC_ERR_TIMEOUT: return "device-side wait timed out";
    case VC_ERR_SCRATCH_LIMIT: return "problem needs more scratch than the built-in array of vc_prep_noalloc holds";
  }
  return "unknown status";
}

}  // extern "C"
