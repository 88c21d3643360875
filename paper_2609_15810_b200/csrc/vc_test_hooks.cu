// Test hooks that run a piece of the attention kernels' arithmetic on its own.
#include "vc_internal.h"
#include "vc_sm100.cuh"

namespace vc {
namespace {

using namespace sm100;

// The ExpCast-FP8 code (Eq. 7) formed exactly as in the softmax stage of the attention kernels:
// per tile fa = cs / 16 and fb = (120 + beta - 8 m) / 128, then expcast_codes4 on four scores.
__global__ void expcast_codes_kernel(const float* __restrict__ s, int64_t n4, float cs, float m, float code_off,
                                     uint32_t* __restrict__ codes) {
  const float fa = cs * 0.0625f, fb = (code_off - 8.0f * m) * 0.0078125f;
  const uint64_t fa2 = pack_f32x2(fa, fa), fb2 = pack_f32x2(fb, fb);
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (int64_t)gridDim.x * blockDim.x) {
    const uint4 v = reinterpret_cast<const uint4*>(s)[i];
    codes[i] = expcast_codes4(v.x, v.y, v.z, v.w, fa2, fb2);
  }
}

}  // namespace
}  // namespace vc

extern "C" vc_status vc_test_expcast_codes(const float* s, int64_t n, float cs, float m, float beta, uint8_t* codes, void* stream) {
  if (n < 0 || (n & 3) || !(cs > 0.f)) return VC_ERR_INVALID_ARG;
  if (n == 0) return VC_OK;
  if (!s || !codes || (((uintptr_t)s | (uintptr_t)codes) & 15)) return VC_ERR_INVALID_ARG;
  const int64_t n4 = n / 4;
  const int blocks = (int)((n4 + 255) / 256 < 4096 ? (n4 + 255) / 256 : 4096);
  vc::expcast_codes_kernel<<<blocks, 256, 0, (cudaStream_t)stream>>>(s, n4, cs, m, 120.0f + (beta != 0.f ? beta : -0.35f),
                                                                     reinterpret_cast<uint32_t*>(codes));
  vc::count_launches(1);
  return cudaGetLastError() == cudaSuccess ? VC_OK : VC_ERR_CUDA;
}
