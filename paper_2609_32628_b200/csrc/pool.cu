// Kernel 1: spatial-tile reorder + 2D average / max pooling of Q and K into per-block draft tokens
// (Eq. "v2-descriptors"; padding of ragged edge tiles excluded, App. C.1), plus the statistics the quantisers
// need before they can run: per-head max|Q|, max|K|, max|V| and per-(head, channel) max|V| (App. C.3).
//
// One CTA per (block, head).  A block is an 8 x 8 tile of one frame: each of its 8 tile rows is 8 consecutive
// tokens, i.e. 8*d*2 contiguous bytes in the raster tensor, so 16-byte loads of a tile row are fully coalesced.
// HBM-bound: reads Q, K, V once (3*N*d*2 bytes per head), writes 4*R*d*4 bytes.
//
// Sums are carried in fp64: a sum of at most 64 bf16 values is exact there, so the fp32 descriptor equals the
// correctly rounded mean regardless of summation order.
#include "da2_internal.cuh"

namespace da2 {

namespace {

__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

template <int D>
__global__ void __launch_bounds__(256) pool_kernel(Params p, const __nv_bfloat16 *__restrict__ q,
                                                   const __nv_bfloat16 *__restrict__ k,
                                                   const __nv_bfloat16 *__restrict__ v) {
  constexpr int CPR = D / 8;          // 16-byte chunks per token row
  constexpr int TP = 256 / CPR;       // token rows per pass
  constexpr int PASSES = kSlots / TP;
  const int a = blockIdx.x, bh = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int cidx = tid % CPR, tsub = tid / CPR;
  const unsigned long long mask = block_valid_mask(p, a);
  const int n_valid = __popcll(mask);
  const size_t head_off = (size_t)bh * p.Ntot * D;

  double sq[8], sk[8];
  float mq[8], mk[8], av[8];
  float aq = 0.f, ak = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) { sq[i] = 0.0; sk[i] = 0.0; mq[i] = -INFINITY; mk[i] = -INFINITY; av[i] = 0.f; }

  // all loads of the thread are issued before the first is used (a padding slot reads slot 0's row and is ignored)
  uint4 xq[PASSES], xk[PASSES], xv[PASSES];
#pragma unroll
  for (int ps = 0; ps < PASSES; ++ps) {
    const int j = ps * TP + tsub;
    const int js = ((mask >> j) & 1ull) ? j : 0;
    const size_t off = head_off + (size_t)slot_token(p, a, js) * D + cidx * 8;
    xq[ps] = *reinterpret_cast<const uint4 *>(q + off);
    xk[ps] = *reinterpret_cast<const uint4 *>(k + off);
    xv[ps] = *reinterpret_cast<const uint4 *>(v + off);
  }
#pragma unroll
  for (int ps = 0; ps < PASSES; ++ps) {
    const int j = ps * TP + tsub;
    if ((mask >> j) & 1ull) {
      const uint32_t wq[4] = {xq[ps].x, xq[ps].y, xq[ps].z, xq[ps].w}, wk[4] = {xk[ps].x, xk[ps].y, xk[ps].z, xk[ps].w},
                     wv[4] = {xv[ps].x, xv[ps].y, xv[ps].z, xv[ps].w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        float f0 = bf16lo(wq[i]), f1 = bf16hi(wq[i]);
        sq[2 * i] += (double)f0; sq[2 * i + 1] += (double)f1;
        mq[2 * i] = fmaxf(mq[2 * i], f0); mq[2 * i + 1] = fmaxf(mq[2 * i + 1], f1);
        aq = fmaxf(aq, fmaxf(fabsf(f0), fabsf(f1)));
        f0 = bf16lo(wk[i]); f1 = bf16hi(wk[i]);
        sk[2 * i] += (double)f0; sk[2 * i + 1] += (double)f1;
        mk[2 * i] = fmaxf(mk[2 * i], f0); mk[2 * i + 1] = fmaxf(mk[2 * i + 1], f1);
        ak = fmaxf(ak, fmaxf(fabsf(f0), fabsf(f1)));
        f0 = fabsf(bf16lo(wv[i])); f1 = fabsf(bf16hi(wv[i]));
        av[2 * i] = fmaxf(av[2 * i], f0); av[2 * i + 1] = fmaxf(av[2 * i + 1], f1);
      }
    }
  }
  // combine the token rows that share a warp (lanes cidx, cidx+CPR, ...)
#pragma unroll
  for (int off = 16; off >= CPR; off >>= 1) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      sq[i] += __shfl_xor_sync(0xffffffffu, sq[i], off);
      sk[i] += __shfl_xor_sync(0xffffffffu, sk[i], off);
      mq[i] = fmaxf(mq[i], __shfl_xor_sync(0xffffffffu, mq[i], off));
      mk[i] = fmaxf(mk[i], __shfl_xor_sync(0xffffffffu, mk[i], off));
      av[i] = fmaxf(av[i], __shfl_xor_sync(0xffffffffu, av[i], off));
    }
  }
  __shared__ double s_sum[2][8][D];
  __shared__ float s_max[3][8][D];
  __shared__ float s_amax[2][8];
  if (lane < CPR) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      s_sum[0][warp][cidx * 8 + i] = sq[i];
      s_sum[1][warp][cidx * 8 + i] = sk[i];
      s_max[0][warp][cidx * 8 + i] = mq[i];
      s_max[1][warp][cidx * 8 + i] = mk[i];
      s_max[2][warp][cidx * 8 + i] = av[i];
    }
  }
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) {
    aq = fmaxf(aq, __shfl_xor_sync(0xffffffffu, aq, off));
    ak = fmaxf(ak, __shfl_xor_sync(0xffffffffu, ak, off));
  }
  if (lane == 0) { s_amax[0][warp] = aq; s_amax[1][warp] = ak; }
  __syncthreads();
  if (tid < D) {
    double tq = 0.0, tk = 0.0;
    float xq = -INFINITY, xk = -INFINITY, xv = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) {
      tq += s_sum[0][w][tid]; tk += s_sum[1][w][tid];
      xq = fmaxf(xq, s_max[0][w][tid]); xk = fmaxf(xk, s_max[1][w][tid]); xv = fmaxf(xv, s_max[2][w][tid]);
    }
    const size_t o = ((size_t)bh * p.R + a) * D + tid;
    p.desc[0][o] = (float)(tq / (double)n_valid);
    p.desc[1][o] = xq;
    p.desc[2][o] = (float)(tk / (double)n_valid);
    p.desc[3][o] = xk;
    // non-negative floats order like their bit patterns
    atomicMax(&p.vmax[(size_t)bh * D + tid], __float_as_uint(xv));
    // head maximum of |V| from the channel maxima: reduce within the warp first
    float hv = xv;
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) hv = fmaxf(hv, __shfl_xor_sync(0xffffffffu, hv, off));
    if (lane == 0) atomicMax(&p.amax[bh * 4 + 2], __float_as_uint(hv));
  }
  if (tid == 0) {
    float tq = 0.f, tk = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) { tq = fmaxf(tq, s_amax[0][w]); tk = fmaxf(tk, s_amax[1][w]); }
    atomicMax(&p.amax[bh * 4 + 0], __float_as_uint(tq));
    atomicMax(&p.amax[bh * 4 + 1], __float_as_uint(tk));
  }
}

// Derived scales (App. C.3): NVFP4 per-tensor scale g_X = amax_X / 2688 (1 for an all-zero head), and the E4M3
// per-channel value scale delta_c = max_v |V_vc| / 2.25 (0 marks an all-zero channel).
__global__ void finalize_stats_kernel(Params p) {
  const int bh = blockIdx.x;
  for (int i = threadIdx.x; i < p.d; i += blockDim.x)
    p.dv8[(size_t)bh * p.d + i] = __fdiv_rn(__uint_as_float(p.vmax[(size_t)bh * p.d + i]), 2.25f);
  if (threadIdx.x < 3) {
    const float am = __uint_as_float(p.amax[bh * 4 + threadIdx.x]);
    p.gscale[bh * 4 + threadIdx.x] = am > 0.f ? __fdiv_rn(am, 2688.0f) : 1.0f;
  }
}

}  // namespace

cudaError_t launch_pool(const Params &p, const __nv_bfloat16 *q, const __nv_bfloat16 *k, const __nv_bfloat16 *v,
                        cudaStream_t st, int *launches) {
  dim3 grid(p.R, p.BH);
  if (p.d == 128) pool_kernel<128><<<grid, 256, 0, st>>>(p, q, k, v);
  else pool_kernel<64><<<grid, 256, 0, st>>>(p, q, k, v);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  finalize_stats_kernel<<<p.BH, 128, 0, st>>>(p);
  *launches += 2;
  return cudaGetLastError();
}

}  // namespace da2
