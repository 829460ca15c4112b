// Measurement aid, not part of the attention path: back-to-back tcgen05.mma instructions of one kind on
// operands that stay resident in shared / tensor memory, one CTA per SM, so that the benchmark can state the
// tensor-core rate this GPU actually sustains for each operand format the attention kernels use
// (kind::f16 BF16 for the rank-one seed of Eq. 11, kind::mxf4nvf4 block-scaled FP4 for Q K^T,
// kind::f8f6f4 E4M3 for P V with A in tensor memory).  The caller times the launch with CUDA events.
#include <cuda_runtime.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace mpfa {
namespace {

constexpr uint32_t PK_A = 0;                 // 128 rows x 128 bytes
constexpr uint32_t PK_B = 16384;             // up to 256 rows x 128 bytes
constexpr uint32_t PK_SF = PK_B + 32768;     // 4 scale-factor atoms of 512 bytes
constexpr uint32_t PK_BAR = PK_SF + 2048;
constexpr uint32_t PK_SMEM = PK_BAR + 64 + 1024;

constexpr uint32_t TM_D = 0, TM_SFA = 256, TM_SFB = 272, TM_A = 320;

__global__ void __launch_bounds__(128, 1) mma_peak_kernel(int kind, int n_cols, int iters, int32_t *status) {
  extern __shared__ uint8_t pk_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(pk_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + PK_BAR + 16);
  const uint32_t bar = sbase + PK_BAR;
  // operand bytes: every byte in 0x20..0x5F - finite in E4M3 and UE4M3, small positive in BF16, any E2M1 pair
  for (uint32_t i = tid; i < (PK_SF + 2048) / 4; i += 128) {
    const uint32_t x = i * 2654435761u;
    reinterpret_cast<uint32_t *>(smem)[i] = ((x >> 7) & 0x3F3F3F3Fu) + 0x20202020u;
  }
  if (tid == 0) {
    mbar_init(bar, 1);
    mbar_init_fence();
  }
  fence_proxy_async_smem();
  if (warp == 0) {
    tmem_alloc(smem_u32(tmem_slot), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tm = *tmem_slot;
  if (warp == 0) {
    if (elect_one()) {
      // scale factors and the tensor-memory A operand: any finite bytes will do
      const uint64_t d_sf = smem_desc(sbase + PK_SF, 0, 128, SWZ_NONE);
      for (int a = 0; a < 4; ++a) tmem_cp_32x128b_warpx4(tm + TM_SFA + 4 * a, d_sf + (uint64_t)((512 * a) >> 4));
      for (int a = 0; a < 4; ++a) tmem_cp_32x128b_warpx4(tm + TM_SFB + 4 * a, d_sf + (uint64_t)((512 * a) >> 4));
      for (int a = 0; a < 8; ++a) tmem_cp_32x128b_warpx4(tm + TM_A + 4 * a, d_sf + (uint64_t)((512 * (a & 3)) >> 4));
      const uint64_t d_a128 = smem_desc(sbase + PK_A, 16, 1024, SWZ_128B);   // K-major rows of 128 bytes
      const uint64_t d_b128 = smem_desc(sbase + PK_B, 16, 1024, SWZ_128B);
      const uint64_t d_a64 = smem_desc(sbase + PK_A, 16, 512, SWZ_64B);      // K-major rows of 64 bytes (FP4, K = 128)
      const uint64_t d_b64 = smem_desc(sbase + PK_B, 16, 512, SWZ_64B);
      const uint32_t id_bf16 = idesc_bf16(128, n_cols, 0, 0);
      const uint32_t id_fp8 = idesc_e4m3(128, n_cols, 0, 0);
      const uint32_t id_fp4 = idesc_nvfp4(128, n_cols);
      for (int it = 0; it < iters; ++it) {
        const uint32_t acc = it > 0 ? 1u : 0u;
        if (kind == 0) {
#pragma unroll
          for (int k = 0; k < 4; ++k) mma_bf16_ss(tm + TM_D, d_a128 + 2 * k, d_b128 + 2 * k, id_bf16, acc | (k > 0));
        } else if (kind == 1) {
#pragma unroll
          for (int k = 0; k < 4; ++k) mma_e4m3_ss(tm + TM_D, d_a128 + 2 * k, d_b128 + 2 * k, id_fp8, acc | (k > 0));
        } else if (kind == 2) {
#pragma unroll
          for (int k = 0; k < 4; ++k) mma_e4m3_ts(tm + TM_D, tm + TM_A + 8 * k, d_b128 + 2 * k, id_fp8, acc | (k > 0));
        } else {
#pragma unroll
          for (int k = 0; k < 4; ++k)
            mma_nvfp4_ss(tm + TM_D, d_a64 + 2 * (k & 1), d_b64 + 2 * (k & 1), id_fp4, tm + TM_SFA + 4 * (k & 1),
                         tm + TM_SFB + 4 * (k & 1), acc | (k > 0));
        }
      }
      mma_commit(bar);
    }
    __syncwarp();
    // bounded wait for the last MMA (about 10 s of SM clock; the loop itself is a few milliseconds)
    const long long t0 = clock64();
    bool done = false;
    while (!(done = mbar_try_wait_hint(bar, 0, 100000u)))
      if (clock64() - t0 > 20000000000ll) break;
    if (!done && (tid & 31) == 0) atomicOr(status, MPFA_DEV_TIMEOUT);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tm, 512);
}

}  // namespace
}  // namespace mpfa

using namespace mpfa;

extern "C" mpfa_status mpfa_bench_mma_peak(int kind, int n_cols, int iters, int32_t *device_status, void *stream) {
  if (kind < 0 || kind > 3 || (n_cols != 128 && n_cols != 256) || iters <= 0 || iters > (1 << 22) || !device_status)
    return MPFA_ERR_INVALID_ARG;
  mpfa_status rc = check_arch();
  if (rc != MPFA_OK) return rc;
  int dev = 0, n_sm = 0;
  MPFA_CUDA_OK(cudaGetDevice(&dev));
  MPFA_CUDA_OK(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev));
  // more than half of an SM's shared memory per CTA: never two CTAs on one SM (the second would sit in the
  // tensor-memory allocation until the first has finished)
  constexpr int LAUNCH_SMEM = 120 * 1024;
  static_assert(LAUNCH_SMEM >= (int)PK_SMEM, "shared memory");
  MPFA_CUDA_OK(cudaFuncSetAttribute(mma_peak_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, LAUNCH_SMEM));
  mma_peak_kernel<<<n_sm, 128, LAUNCH_SMEM, static_cast<cudaStream_t>(stream)>>>(kind, n_cols, iters, device_status);
  MPFA_LAUNCH_OK();
  return MPFA_OK;
}

extern "C" double mpfa_bench_mma_flops(int kind, int n_cols, int iters) {
  const double k = kind == 0 ? 16.0 : (kind == 3 ? 64.0 : 32.0);
  return 4.0 * (double)iters * 2.0 * 128.0 * (double)n_cols * k;   // per CTA
}
