// Tensor-core microbenchmark: back-to-back tcgen05.mma of one kind and shape on every SM, operands in shared memory,
// accumulators in tensor memory.  It gives this GPU's own per-kind peaks (bf16, INT8, E4M3, block-scaled NVFP4) at the
// tile shapes the attention kernel can use (M = 128, N = 64 / 128 / 256), which is what the roofline of the phased
// attention kernel is quoted against beside the nominal figures.  Diagnostic only: nothing on the attention path
// calls it.
#include "da2_internal.cuh"
#include "tc05.cuh"

namespace da2 {

namespace {

constexpr int kPeakThreads = 128;
constexpr uint32_t kPeakSmem = 16384 + 32768 + 2048;  // A: 128 rows x 128 B, B: 256 rows x 128 B, scale atoms

// kind: 0 bf16 (K = 16 per instruction), 1 INT8 (K = 32), 2 E4M3 (K = 32), 3 NVFP4 block-scaled (K = 64)
template <int KIND>
__global__ void __launch_bounds__(kPeakThreads, 1) mma_peak_kernel(int n, int iters, long long *out) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ uint32_t s_tmem;
  __shared__ uint64_t s_bar;
  __shared__ int s_fail;
  const int tid = threadIdx.x, warp = tid >> 5;
  for (uint32_t i = tid; i < kPeakSmem / 4; i += kPeakThreads) reinterpret_cast<uint32_t *>(smem)[i] = 0;
  if (warp == 0) {
    tc::tmem_alloc(&s_tmem, 512);
    tc::tmem_relinquish();
  }
  if (tid == 32) {
    tc::mbar_init(&s_bar, 1);
    tc::fence_barrier_init();
    s_fail = 0;
  }
  tc::fence_async_smem();
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tmem = s_tmem;
  if (warp == 1) {
    // K-major images without swizzle: 16-byte chunk (kc, r) at (kc * rows + r) * 16; one instruction reads two chunks
    const uint32_t a_addr = tc::smem_u32(smem), b_addr = a_addr + 16384, sf_addr = b_addr + 32768;
    const uint64_t ad = tc::smem_desc(a_addr, 128 * 16, 128), bd = tc::smem_desc(b_addr, (uint32_t)n * 16, 128);
    const uint32_t a_step = (2 * 128 * 16) >> 4, b_step = (2 * (uint32_t)n * 16) >> 4;
    const uint32_t idesc = KIND == 0 ? tc::idesc_bf16(n) : KIND == 1 ? tc::idesc_i8(n)
                         : KIND == 2 ? tc::idesc_e4m3(n) : tc::idesc_nvfp4(n);
    const uint32_t t_sfa = tmem + 480, t_sfb = tmem + 488;
    if (KIND == 3 && tc::elect_one()) {
      tc::tmem_cp_sf(t_sfa, tc::smem_desc(sf_addr, 128, 128));
      tc::tmem_cp_sf(t_sfb, tc::smem_desc(sf_addr + 512, 128, 128));
      tc::tmem_cp_sf(t_sfb + 4, tc::smem_desc(sf_addr + 1024, 128, 128));
    }
    __syncwarp();
    const long long t0 = clock64();
    // warp-uniform loop, one elected lane issues: two accumulators used alternately, and per accumulator four
    // instructions that walk a 128-byte reduction row, as one score tile does
    const uint32_t d1 = tmem + (n < 256 ? (uint32_t)n : 0u);
    for (int it = 0; it < iters; it += 2) {
      if (tc::elect_one()) {
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const uint32_t d = u ? d1 : tmem;
#pragma unroll
          for (int ks = 0; ks < 4; ++ks) {
            const uint64_t a = ad + ks * a_step, b = bd + ks * b_step;
            if (KIND == 0) tc::mma_f16(d, a, b, idesc, ks > 0);
            else if (KIND == 1) tc::mma_i8(d, a, b, idesc, ks > 0);
            else if (KIND == 2) tc::mma_f8f6f4(d, a, b, idesc, ks > 0);
            else tc::mma_nvfp4(d, a, b, idesc, ks > 0, t_sfa, t_sfb);
          }
        }
      }
      __syncwarp();
    }
    if (tc::elect_one()) tc::mma_commit(&s_bar);
    __syncwarp();
    if (!tc::mbar_wait(&s_bar, 0)) s_fail = 1;  // bounded
    const long long t1 = clock64();
    if (blockIdx.x == 0 && (tid & 31) == 0) {
      out[0] = t1 - t0;
      out[1] = (long long)((iters + 1) / 2) * 8;
      out[2] = s_fail;
    }
  }
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 0) tc::tmem_dealloc(tmem, 512);
}

}  // namespace

}  // namespace da2

extern "C" da2_status_t da2_tcgen05_peak(int32_t kind, int32_t n, int32_t iters, int32_t ctas, void *out_dev,
                                         void *stream) {
  if (kind < 0 || kind > 3 || (n != 64 && n != 128 && n != 256) || iters < 1 || iters > (1 << 20) || ctas < 1 ||
      ctas > 4096 || !out_dev)
    return DA2_ERR_INVALID_ARG;
  auto launch = [&](auto kernel) -> cudaError_t {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)da2::kPeakSmem);
    if (e != cudaSuccess) return e;
    kernel<<<ctas, da2::kPeakThreads, da2::kPeakSmem, (cudaStream_t)stream>>>(n, iters, (long long *)out_dev);
    return cudaGetLastError();
  };
  const cudaError_t e = kind == 0 ? launch(da2::mma_peak_kernel<0>) : kind == 1 ? launch(da2::mma_peak_kernel<1>)
                      : kind == 2 ? launch(da2::mma_peak_kernel<2>) : launch(da2::mma_peak_kernel<3>);
  return e == cudaSuccess ? DA2_OK : DA2_ERR_CUDA;
}
