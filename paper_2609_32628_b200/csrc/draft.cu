// Kernel 2, first half: low-resolution draft logits (Def. 3.1, Eq. "v2-draft").
//   logits[0][bh][a][b] = scale * Qavg_a . Kavg_b      logits[1][bh][a][b] = scale * Qmax_a . Kmax_b
// The row softmaxes, their mixture and the ranking follow in rank.cu.
//
// The ranking compares scores to about 1e-5 relative and a softmax turns an ABSOLUTE logit error into a RELATIVE
// score error, so the contraction accumulates in fp64 (products of fp32 descriptors are exact there) and only the
// final logit is rounded to fp32; with large logits (outlier channels) fp32 accumulation alone would already move
// scores by 1e-4.  It is a small GEMM: 4*R*R*d flops per head, against 4*64*64*d flops per retained block pair in
// the attention kernel.
// The plain fp64 pipe sustains about half of what the fp64 tensor-core path does on this part, so the products run as
// mma.sync m8n8k4 (fp64 in, fp64 accumulate): 128 x 64 output tile per CTA, 32 x 32 per warp (4 x 4 fragments), K
// panels of 16 channels in shared memory.  The descriptors are widened to fp64 once, when a panel is staged.
#include "da2_internal.cuh"

namespace da2 {

namespace {

constexpr int TM = 128, TN = 64, TK = 16;
constexpr int LDA = TM + 4, LDB = TN + 4;  // row strides = 4 mod 16 doubles: the 16 lanes of a half warp hit 16 bank pairs

__device__ __forceinline__ void dmma(double (&c)[2], double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
               : "+d"(c[0]), "+d"(c[1])
               : "d"(a), "d"(b));
}

__global__ void __launch_bounds__(256) draft_logits_kernel(Params p) {
  const int which = blockIdx.z & 1, bh = blockIdx.z >> 1;
  const float *__restrict__ Qd = p.desc[which] + (size_t)bh * p.R * p.d;       // Qavg or Qmax
  const float *__restrict__ Kd = p.desc[2 + which] + (size_t)bh * p.R * p.d;   // Kavg or Kmax
  float *__restrict__ out = p.logits[which] + (size_t)bh * p.R * p.R;
  const int a0 = blockIdx.y * TM, b0 = blockIdx.x * TN;
  __shared__ __align__(16) double As[TK][LDA];  // [channel][query block]
  __shared__ __align__(16) double Bs[TK][LDB];  // [channel][key block]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int wm = (warp & 3) * 32, wn = (warp >> 2) * 32;  // warp tile origin inside the CTA tile
  const int fr = lane >> 2, fc = lane & 3;                // fragment row (or column of B) and channel inside a k4 step
  double acc[4][4][2];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) { acc[i][j][0] = 0.0; acc[i][j][1] = 0.0; }

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
    for (int k4 = 0; k4 < TK; k4 += 4) {
      double af[4], bf[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) af[i] = As[k4 + fc][wm + i * 8 + fr];
#pragma unroll
      for (int j = 0; j < 4; ++j) bf[j] = Bs[k4 + fc][wn + j * 8 + fr];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) dmma(acc[i][j], af[i], bf[j]);
    }
  }
  // accumulator fragment: row = lane / 4, columns 2 * (lane % 4) and + 1
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int a = a0 + wm + i * 8 + fr;
    if (a >= p.R) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int b = b0 + wn + j * 8 + fc * 2;
      if (b < p.R) out[(size_t)a * p.R + b] = (float)((double)p.scale * acc[i][j][0]);
      if (b + 1 < p.R) out[(size_t)a * p.R + b + 1] = (float)((double)p.scale * acc[i][j][1]);
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
