// Measurement aid: the tensor-core rate the attention kernels are held against, measured on the
// GPU at hand instead of derived from a bf16 figure and a nominal ratio.  Every SM issues a long
// run of back-to-back tcgen05.mma of ONE kind on tiles that stay resident in shared memory
// (accumulating into tensor memory, nothing loaded or stored inside the run), which is the
// work the attention kernels' two products consist of with everything else taken away:
//   kind 8   kind::f8f6f4, E4M3 x E4M3, M128 N128 K32          (the 8-bit products)
//   kind 4   kind::mxf4nvf4.block16, E2M1 under UE4M3 factors, M128 N128 K64   (the 4-bit products)
// The result is a ceiling for a kernel that does nothing but these MMAs; the bench reports the
// attention kernels as a fraction of it beside the bf16-derived figures.
#include "vc_attn_shared.cuh"
#include "vc_internal.h"
#include "vc_sm100.cuh"

namespace vc {
namespace {

using namespace sm100;

template <int KIND>
__global__ void __launch_bounds__(128) mma_peak_kernel(long long* cycles, int groups) {
  extern __shared__ unsigned char raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
  constexpr int kRow = KIND == 8 ? 128 : 64;       // bytes per operand row: 128 E4M3 or 128 E2M1 channels
  unsigned char* sA = smem;                        // 128 rows
  unsigned char* sB = smem + 128 * kRow;           // 128 rows
  unsigned char* sSf = sB + 128 * kRow;            // one 512-byte chunk of scale factors (kind 4)
  __shared__ uint64_t bar;
  __shared__ uint32_t slot;
  // E4M3 1.0 bytes, resp. E2M1 (1.0, 1.0) bytes, and factor 1.0: finite operands, exact sums
  for (int i = threadIdx.x; i < 2 * 128 * kRow; i += 128) smem[i] = KIND == 8 ? 0x38 : 0x22;
  for (int i = threadIdx.x; i < 512; i += 128) sSf[i] = 0x38;
  if (threadIdx.x == 0) { mbar_init(&bar, 1); mbar_fence_init(); }
  if (threadIdx.x < 32) { tmem_alloc<512>(&slot); tmem_relinquish(); }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = slot;
  if (threadIdx.x == 0) {
    const uint64_t da = smem_desc_kmajor(smem_u32(sA), kRow), db = smem_desc_kmajor(smem_u32(sB), kRow);
    constexpr uint32_t SF_COL = 256;
    if (KIND == 4) {
      tmem_cp_sf(tmem + SF_COL, smem_desc_sf_chunk(smem_u32(sSf)));
      tmem_cp_sf(tmem + SF_COL + 4, smem_desc_sf_chunk(smem_u32(sSf)));
    }
    const uint32_t idesc = KIND == 8 ? idesc_e4m3(128, 128) : idesc_nvfp4(128, 128);
    const long long t0 = clock64();
    for (int g = 0; g < groups; ++g) {             // a group = one 128 x 128 x 128 product, two accumulators in turn
      const uint32_t acc = tmem + 128 * (g & 1);
      if (KIND == 8) {
#pragma unroll
        for (int k = 0; k < 4; ++k) mma_f8_ss(acc, da + 2 * k, db + 2 * k, idesc, (g > 1) | (k > 0));
      } else {
#pragma unroll
        for (int k = 0; k < 2; ++k) mma_nvfp4_ss(acc, da + 2 * k, db + 2 * k, idesc, (g > 1) | (k > 0), tmem + SF_COL, tmem + SF_COL + 4);
      }
    }
    mma_commit(&bar);
    const bool ok = mbar_wait(&bar, 0, attn::kDrainLimit);     // bounded; the MMAs have completed
    const long long t1 = clock64();
    if (blockIdx.x == 0) cycles[0] = ok ? t1 - t0 : -1;
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x < 32) tmem_dealloc<512>(tmem);
}

}  // namespace
}  // namespace vc

using namespace vc;

extern "C" vc_status vc_mma_peak(int32_t kind, int32_t groups, void* scratch, double* tflops, double* mac_per_clk_sm, void* stream) {
  if ((kind != 8 && kind != 4) || groups < 1 || groups > (1 << 20) || !scratch || ((uintptr_t)scratch & 7) || !tflops || !mac_per_clk_sm)
    return VC_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
    return VC_ERR_CUDA;
  long long* d_cycles = reinterpret_cast<long long*>(scratch);
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  vc_status st = VC_ERR_CUDA;
  const size_t smem = 1024 + 2 * 128 * 128 + 512;
  if ((kind == 8 ? cudaFuncSetAttribute(mma_peak_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)
                 : cudaFuncSetAttribute(mma_peak_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) == cudaSuccess &&
      cudaEventCreate(&e0) == cudaSuccess && cudaEventCreate(&e1) == cudaSuccess) {
    auto launch = [&](int n) {
      if (kind == 8) mma_peak_kernel<8><<<sms, 128, smem, s>>>(d_cycles, n);
      else mma_peak_kernel<4><<<sms, 128, smem, s>>>(d_cycles, n);
    };
    launch(groups);                                            // warm-up
    cudaEventRecord(e0, s);
    launch(groups);
    cudaEventRecord(e1, s);
    count_launches(2);
    long long h = 0;
    float ms = 0.f;
    if (cudaEventSynchronize(e1) == cudaSuccess && cudaEventElapsedTime(&ms, e0, e1) == cudaSuccess &&
        cudaMemcpy(&h, d_cycles, 8, cudaMemcpyDeviceToHost) == cudaSuccess && cudaGetLastError() == cudaSuccess) {
      if (h <= 0 || ms <= 0.f) st = VC_ERR_TIMEOUT;
      else {
        const double macs = (double)groups * 128.0 * 128.0 * 128.0;   // per SM
        *tflops = 2.0 * macs * sms / (ms * 1e-3) / 1e12;
        *mac_per_clk_sm = macs / (double)h;
        st = VC_OK;
      }
    }
  }
  if (e0) cudaEventDestroy(e0);
  if (e1) cudaEventDestroy(e1);
  return st;
}
