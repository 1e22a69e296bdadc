// Kernel 2, first half: low-resolution draft logits (Def. 3.1, Eq. "v2-draft").
//   logits[0][bh][a][b] = scale * Qavg_a . Kavg_b      logits[1][bh][a][b] = scale * Qmax_a . Kmax_b
// The row softmaxes, their mixture and the ranking follow in rank.cu.
//
// The ranking compares scores to about 1e-5 relative and a softmax turns an ABSOLUTE logit error into a RELATIVE
// score error, so the contraction accumulates in fp64 (products of fp32 descriptors are exact there) and only the
// final logit is rounded to fp32; with large logits (outlier channels) fp32 accumulation alone would already move
// scores by 1e-4.  It is a small GEMM: 4*R*R*d flops per head, against 4*64*64*d flops per retained block pair in
// the attention kernel, so the fp64 rate is not a concern.
// 64 x 64 output tile per CTA, 4 x 4 register tile per thread, K panel of 16 channels in shared memory.
#include "da2_internal.cuh"

namespace da2 {

namespace {

constexpr int TM = 64, TN = 64, TK = 16;

__global__ void __launch_bounds__(256) draft_logits_kernel(Params p) {
  const int which = blockIdx.z & 1, bh = blockIdx.z >> 1;
  const float *__restrict__ Qd = p.desc[which] + (size_t)bh * p.R * p.d;       // Qavg or Qmax
  const float *__restrict__ Kd = p.desc[2 + which] + (size_t)bh * p.R * p.d;   // Kavg or Kmax
  float *__restrict__ out = p.logits[which] + (size_t)bh * p.R * p.R;
  const int a0 = blockIdx.y * TM, b0 = blockIdx.x * TN;
  __shared__ float As[TK][TM + 4];
  __shared__ float Bs[TK][TN + 4];
  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;  // thread tile: rows ty*4.., cols tx*4..
  double acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.0;

  // loader mapping: 64 rows x 16 channels = 256 float4 quarters -> one float4 per thread per matrix
  const int lr = tid >> 2, lc = (tid & 3) * 4;
  for (int c0 = 0; c0 < p.d; c0 += TK) {
    float4 xa = make_float4(0.f, 0.f, 0.f, 0.f), xb = xa;
    if (a0 + lr < p.R) xa = *reinterpret_cast<const float4 *>(Qd + (size_t)(a0 + lr) * p.d + c0 + lc);
    if (b0 + lr < p.R) xb = *reinterpret_cast<const float4 *>(Kd + (size_t)(b0 + lr) * p.d + c0 + lc);
    __syncthreads();
    As[lc + 0][lr] = xa.x; As[lc + 1][lr] = xa.y; As[lc + 2][lr] = xa.z; As[lc + 3][lr] = xa.w;
    Bs[lc + 0][lr] = xb.x; Bs[lc + 1][lr] = xb.y; Bs[lc + 2][lr] = xb.z; Bs[lc + 3][lr] = xb.w;
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < TK; ++kk) {
      const float4 av = *reinterpret_cast<const float4 *>(&As[kk][ty * 4]);
      const float4 bv = *reinterpret_cast<const float4 *>(&Bs[kk][tx * 4]);
      const double ar[4] = {av.x, av.y, av.z, av.w}, br[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fma(ar[i], br[j], acc[i][j]);
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int a = a0 + ty * 4 + i;
    if (a >= p.R) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int b = b0 + tx * 4 + j;
      if (b < p.R) out[(size_t)a * p.R + b] = (float)((double)p.scale * acc[i][j]);
    }
  }
}

}  // namespace

cudaError_t launch_draft(const Params &p, cudaStream_t st, int *launches) {
  dim3 grid((p.R + TN - 1) / TN, (p.R + TM - 1) / TM, p.BH * 2);
  draft_logits_kernel<<<grid, 256, 0, st>>>(p);
  *launches += 1;
  return cudaGetLastError();
}

}  // namespace da2
