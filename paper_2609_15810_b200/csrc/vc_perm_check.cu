// Validator of the token-group permutation (VC_FLAG_CHECK_PERM).  Eq. 3 needs pi to be a
// permutation of [0, N) per (batch, head).  The gathers of the preprocessing kernels clamp every
// entry into [0, N), so a bad pi can never become a bad address; this kernel is what tells the
// caller: one bit per (head, token value), an entry out of range or seen twice sets a code in
// the status word, which vc_poll_status returns as VC_ERR_INVALID_ARG.
#include "vc_internal.h"

namespace vc {
namespace {

// Every entry inside [0, N) and none twice.
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

}  // namespace vc
