// Kernel 2, first half: low-resolution draft logits (Def. 3.1, Eq. "v2-draft").
//   logits[0][bh][a][b] = scale * Qavg_a . Kavg_b      logits[1][bh][a][b] = scale * Qmax_a . Kmax_b
// The row softmaxes, their mixture and the ranking follow in rank.cu.
//
// The ranking compares scores to about 1e-5 relative and a softmax turns an ABSOLUTE logit error into a RELATIVE
// score error, so the contraction accumulates in fp64 (products of fp32 descriptors are exact there) and only the
// final logit is rounded to fp32; with large logits (outlier channels) fp32 accumulation alone would already move
// scores by 1e-4.  It is a small GEMM: 4*R*R*d flops per head, against 4*64*64*d flops per retained block pair in
// the attention kernel, so the fp64 rate is not a concern.
// 128 x 64 output tile per CTA, 8 x 4 register tile per thread, K panel of 16 channels in shared memory.  The
// descriptors are widened to fp64 once, when a panel is staged (a conversion per use would cost more than the
// multiply-add it feeds), and every output sums its channels in ascending order whatever the tiling.
#include "da2_internal.cuh"

namespace da2 {

namespace {

constexpr int TM = 128, TN = 64, TK = 16;

__global__ void __launch_bounds__(256) draft_logits_kernel(Params p) {
  const int which = blockIdx.z & 1, bh = blockIdx.z >> 1;
  const float *__restrict__ Qd = p.desc[which] + (size_t)bh * p.R * p.d;       // Qavg or Qmax
  const float *__restrict__ Kd = p.desc[2 + which] + (size_t)bh * p.R * p.d;   // Kavg or Kmax
  float *__restrict__ out = p.logits[which] + (size_t)bh * p.R * p.R;
  const int a0 = blockIdx.y * TM, b0 = blockIdx.x * TN;
  __shared__ __align__(16) double As[TK][TM + 2];
  __shared__ __align__(16) double Bs[TK][TN + 2];
  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;  // thread tile: rows ty*8.., cols tx*4..
  double acc[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.0;

  // loader mapping: 64 rows x 16 channels = 256 float4 quarters -> one float4 per thread per 64 rows
  const int lr = tid >> 2, lc = (tid & 3) * 4;
  for (int c0 = 0; c0 < p.d; c0 += TK) {
    float4 xa0 = make_float4(0.f, 0.f, 0.f, 0.f), xa1 = xa0, xb = xa0;
    if (a0 + lr < p.R) xa0 = *reinterpret_cast<const float4 *>(Qd + (size_t)(a0 + lr) * p.d + c0 + lc);
    if (a0 + 64 + lr < p.R) xa1 = *reinterpret_cast<const float4 *>(Qd + (size_t)(a0 + 64 + lr) * p.d + c0 + lc);
    if (b0 + lr < p.R) xb = *reinterpret_cast<const float4 *>(Kd + (size_t)(b0 + lr) * p.d + c0 + lc);
    __syncthreads();
    As[lc + 0][lr] = xa0.x; As[lc + 1][lr] = xa0.y; As[lc + 2][lr] = xa0.z; As[lc + 3][lr] = xa0.w;
    As[lc + 0][64 + lr] = xa1.x; As[lc + 1][64 + lr] = xa1.y; As[lc + 2][64 + lr] = xa1.z; As[lc + 3][64 + lr] = xa1.w;
    Bs[lc + 0][lr] = xb.x; Bs[lc + 1][lr] = xb.y; Bs[lc + 2][lr] = xb.z; Bs[lc + 3][lr] = xb.w;
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < TK; ++kk) {
      double ar[8], br[4];
#pragma unroll
      for (int i = 0; i < 8; i += 2) {
        const double2 t = *reinterpret_cast<const double2 *>(&As[kk][ty * 8 + i]);
        ar[i] = t.x; ar[i + 1] = t.y;
      }
#pragma unroll
      for (int j = 0; j < 4; j += 2) {
        const double2 t = *reinterpret_cast<const double2 *>(&Bs[kk][tx * 4 + j]);
        br[j] = t.x; br[j + 1] = t.y;
      }
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fma(ar[i], br[j], acc[i][j]);
    }
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int a = a0 + ty * 8 + i;
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
