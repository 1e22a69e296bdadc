// Kernel 3: fused operand preparation.  One pass over Q, K, V reorders every 8 x 8 spatial tile into a contiguous
// block and quantises it to each active format (App. C.3), writing the result directly as the shared-memory image
// the attention kernel streams in (K-major 8 x 16-byte core matrices, V already transposed to [channel][key slot],
// scale factors in the layout the block-scaled tensor-core instruction reads) -- see da2.h for the record layout.
//   INT8  Q/K : one fp32 scale per block, delta = amax/127 + 1e-7, round half away from zero
//   E4M3  V   : per-(head, channel) scale delta_c = max|V_c| / 2.25
//   NVFP4 Q/K : E2M1 with one E4M3 scale per 16 channels; V: per 16 key slots of a channel; per-head scale g_X
//   BF16      : the stored values, reordered only
// Every fp32 operation below is a single correctly rounded operation in the order the format definition gives, so
// codes and scales are reproducible bit for bit.  HBM-bound: reads 3*64*d*2 bytes per block, writes the records.
#include <cuda_fp8.h>

#include "da2_internal.cuh"

namespace da2 {

namespace {

constexpr int NT = 256;

__device__ __forceinline__ float bf16_to_f32(uint16_t b) { return __uint_as_float((uint32_t)b << 16); }

// round half away from zero for |x| < 2^23: adding the largest float below one half (with the sign of x) and truncating
// gives the same integer as roundf for every x in that range (the sum can only round up to the next integer when x
// is at least one half above the integer below it)
__device__ __forceinline__ int round_half_away(float x) { return __float2int_rz(__fadd_rn(x, copysignf(0x1.fffffep-2f, x))); }

__device__ __forceinline__ uint32_t cast_e4m3(float x) {
  return (uint32_t)__nv_cvt_float_to_fp8(x, __NV_SATFINITE, __NV_E4M3);
}

// two floats -> two E2M1 codes, `lo` in bits 3:0 and `hi` in bits 7:4 (round to nearest even, saturating)
__device__ __forceinline__ uint32_t cast_e2m1x2(float lo, float hi) {
  uint16_t r;
  asm("{ .reg .b8 t; cvt.rn.satfinite.e2m1x2.f32 t, %2, %1; mov.b16 %0, {t, 0}; }" : "=h"(r) : "f"(lo), "f"(hi));
  return (uint32_t)r;
}

__device__ __forceinline__ float decode_e4m3(uint32_t c) {
  const __half_raw h = __nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)c, __NV_E4M3);
  return __half2float(*reinterpret_cast<const __half *>(&h));
}

// Correctly rounded x / d for many x and one positive divisor d, without a division per element: with r = RN(1/d),
// q0 = RN(x r), e = x - q0 d (exact in one fused multiply-add) and q = RN(q0 + e r) is the correctly rounded quotient
// (Markstein's division theorem).  Checked exhaustively on the device against the IEEE division for every bf16 x
// with |x| >= 2^-100 and millions of divisors in [2^-60, 2^60], significands of all ones included: the only
// difference is the sign of a zero quotient, which the sign copy restores (d > 0).  For |x| < 2^-100 the residual can
// underflow; the quotient is then below 2^-40 in magnitude either way and every format here encodes it as a signed
// zero.  Divisors outside [2^-60, 2^60] (or not finite) keep the plain division.  da2_selfcheck_quantiser_arithmetic
// repeats the check with these very functions.
struct Divider {
  float d, r;
  bool fast;
  __device__ __forceinline__ float quick(float x) const {
    const float q0 = __fmul_rn(x, r);
    const float e = __fmaf_rn(-q0, d, x);
    return copysignf(__fmaf_rn(e, r, q0), x);
  }
  __device__ __forceinline__ float exact(float x) const { return __fdiv_rn(x, d); }
};
__device__ __forceinline__ Divider make_divider(float d) {
  Divider v;
  v.d = d;
  v.r = __frcp_rn(d);
  v.fast = d >= 8.6736174e-19f && d <= 1.1529215e18f;
  return v;
}

// NVFP4 group of 16 values (Eq. "v2-nvfp4-quantization"): returns the E4M3 scale code, writes 8 bytes of codes
__device__ __forceinline__ uint32_t nvfp4_group(const float (&x)[16], float g, uint32_t (&packed)[2]) {
  float gmax = 0.f;
#pragma unroll
  for (int i = 0; i < 16; ++i) gmax = fmaxf(gmax, fabsf(x[i]));
  const uint32_t sc = cast_e4m3(__fdiv_rn(gmax, __fmul_rn(6.0f, g)));
  const float sigma = decode_e4m3(sc);
  packed[0] = 0; packed[1] = 0;
  if (sigma == 0.f) return sc;  // a group whose encoded scale is zero is encoded as zero
  const Divider dv = make_divider(__fmul_rn(g, sigma));
  if (dv.fast) {
#pragma unroll
    for (int i = 0; i < 8; ++i) packed[i >> 2] |= cast_e2m1x2(dv.quick(x[2 * i]), dv.quick(x[2 * i + 1])) << (8 * (i & 3));
  } else {
#pragma unroll
    for (int i = 0; i < 8; ++i) packed[i >> 2] |= cast_e2m1x2(dv.exact(x[2 * i]), dv.exact(x[2 * i + 1])) << (8 * (i & 3));
  }
  return sc;
}

// POOL: the pass also writes the block's average and max descriptors of Q and K (Eq. "v2-descriptors"), so that a
// call whose quantiser statistics are already known reads Q, K, V from HBM exactly once (Sec. 3.3, "Fused
// quantization and reordering").
template <int D, bool POOL>
__global__ void __launch_bounds__(NT) prep_kernel(Params p, const __nv_bfloat16 *__restrict__ q,
                                                  const __nv_bfloat16 *__restrict__ k,
                                                  const __nv_bfloat16 *__restrict__ v) {
  extern __shared__ __align__(16) uint8_t smem[];
  uint16_t *tq = reinterpret_cast<uint16_t *>(smem);   // [64][D]
  // rows are padded by 16 bytes: threads that read the same channels of consecutive slots then fall on different banks
  constexpr int LD = D + 8;
  uint16_t *tk = tq + kSlots * LD;
  uint16_t *tv = tk + kSlots * LD;
  uint8_t *sf_img = reinterpret_cast<uint8_t *>(tv + kSlots * LD);  // up to 3 atoms (Q or K: D/64, V: 1)
  __shared__ float s_red[2][NT / 32];
  __shared__ float s_delta[2];

  const int a = blockIdx.x, bh = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const unsigned long long mask = block_valid_mask(p, a);
  const size_t head_off = (size_t)bh * p.Ntot * D;
  const size_t blk = (size_t)bh * p.R + a;        // record index in the quantised tiers (video blocks only)
  const size_t blk16 = (size_t)bh * p.Rt + a;     // record index in the 16-bit tier (video and prefix blocks)
  const bool video = a < p.R;                      // prefix blocks only ever run in the 16-bit tier (App. C.1)
  // the regions of the first frame also leave the frame's region table for the attention kernel
  if (bh == 0 && a < p.R_f) {
    if (tid < kSlots) p.region_cell[a * kSlots + tid] = (int)(slot_token(p, a, tid) - p.P);
    if (tid == 0) p.region_mask[a] = mask;
  }

  // stage the three tiles, padding slots as zeros; track max|Q|, max|K| of the block
  float aq = 0.f, ak = 0.f;
  constexpr int CPR = D / 8;
  for (int idx = tid; idx < kSlots * CPR; idx += NT) {
    const int j = idx / CPR, c8 = idx % CPR;
    uint4 xq = make_uint4(0, 0, 0, 0), xk = xq, xv = xq;
    if ((mask >> j) & 1ull) {
      const size_t off = head_off + (size_t)slot_token(p, a, j) * D + c8 * 8;
      xq = *reinterpret_cast<const uint4 *>(q + off);
      xk = *reinterpret_cast<const uint4 *>(k + off);
      xv = *reinterpret_cast<const uint4 *>(v + off);
    }
    *reinterpret_cast<uint4 *>(tq + j * LD + c8 * 8) = xq;
    *reinterpret_cast<uint4 *>(tk + j * LD + c8 * 8) = xk;
    *reinterpret_cast<uint4 *>(tv + j * LD + c8 * 8) = xv;
    const uint32_t wq[4] = {xq.x, xq.y, xq.z, xq.w}, wk[4] = {xk.x, xk.y, xk.z, xk.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      aq = fmaxf(aq, fmaxf(fabsf(__uint_as_float(wq[i] << 16)), fabsf(__uint_as_float(wq[i] & 0xffff0000u))));
      ak = fmaxf(ak, fmaxf(fabsf(__uint_as_float(wk[i] << 16)), fabsf(__uint_as_float(wk[i] & 0xffff0000u))));
    }
  }
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) {
    aq = fmaxf(aq, __shfl_xor_sync(0xffffffffu, aq, o));
    ak = fmaxf(ak, __shfl_xor_sync(0xffffffffu, ak, o));
  }
  if (lane == 0) { s_red[0][warp] = aq; s_red[1][warp] = ak; }
  __syncthreads();
  if (tid < 2) {
    float m = 0.f;
#pragma unroll
    for (int w = 0; w < NT / 32; ++w) m = fmaxf(m, s_red[tid][w]);
    const float delta = __fadd_rn(__fdiv_rn(m, 127.0f), 1e-7f);
    s_delta[tid] = delta;
    if (p.tier_active[1] && video) (tid == 0 ? p.dq8 : p.dk8)[blk] = delta;
  }
  __syncthreads();

  if (POOL && video) {
    // one thread per (tensor, channel): sum and maximum over the valid slots of the staged tile.  A sum of at most
    // 64 bf16 values is exact in fp64, so the mean is correctly rounded whatever the order.
    const int n_valid = __popcll(mask);
    for (int idx = tid; idx < 2 * D; idx += NT) {
      const uint16_t *src = (idx < D ? tq : tk) + (idx % D);
      double sum = 0.0;
      float mx = -INFINITY;
#pragma unroll 8
      for (int j = 0; j < kSlots; ++j) {
        if ((mask >> j) & 1ull) {
          const float x = bf16_to_f32(src[j * LD]);
          sum += (double)x;
          mx = fmaxf(mx, x);
        }
      }
      const size_t o = blk * D + (idx % D);
      p.desc[idx < D ? 0 : 2][o] = (float)(sum / (double)n_valid);
      p.desc[idx < D ? 1 : 3][o] = mx;
    }
  }

  // ------------------------------------------------------------------ tier 2: BF16, reorder only
  if (p.tier_active[2]) {
    uint8_t *qr = p.qrec[2] + blk16 * p.qrec_bytes[2];
    uint8_t *kr = p.kvrec[2] + blk16 * p.kvrec_bytes[2];
    uint8_t *vr = kr + kSlots * D * 2;
    for (int idx = tid; idx < kSlots * D / 8; idx += NT) {  // chunk (kc, r): channels kc*8.. of slot r
      const int kc = idx / kSlots, r = idx % kSlots;
      *reinterpret_cast<uint4 *>(qr + (size_t)idx * 16) = *reinterpret_cast<const uint4 *>(tq + r * LD + kc * 8);
      *reinterpret_cast<uint4 *>(kr + (size_t)idx * 16) = *reinterpret_cast<const uint4 *>(tk + r * LD + kc * 8);
    }
    for (int idx = tid; idx < D * kSlots / 8; idx += NT) {  // chunk (kc, c): slots kc*8.. of channel c
      const int kc = idx / D, c = idx % D;
      uint32_t w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i)
        w[i] = (uint32_t)tv[(kc * 8 + 2 * i) * LD + c] | ((uint32_t)tv[(kc * 8 + 2 * i + 1) * LD + c] << 16);
      *reinterpret_cast<uint4 *>(vr + (size_t)idx * 16) = make_uint4(w[0], w[1], w[2], w[3]);
    }
  }

  // ------------------------------------------------------------------ tier 1: INT8 Q/K, E4M3 V
  if (p.tier_active[1] && video) {
    uint8_t *qr = p.qrec[1] + blk * p.qrec_bytes[1];
    uint8_t *kr = p.kvrec[1] + blk * p.kvrec_bytes[1];
    uint8_t *vr = kr + kSlots * D;
    const Divider dq = make_divider(s_delta[0]), dk = make_divider(s_delta[1]);  // delta >= 1e-7: always in the quick range
    for (int idx = tid; idx < kSlots * D / 16; idx += NT) {  // chunk (kc, r): channels kc*16.. of slot r
      const int kc = idx / kSlots, r = idx % kSlots;
      uint32_t wq[4] = {0, 0, 0, 0}, wk[4] = {0, 0, 0, 0};
      uint32_t xq[8], xk[8];  // 16 bf16 values each, two per word
      *reinterpret_cast<uint4 *>(xq) = *reinterpret_cast<const uint4 *>(tq + r * LD + kc * 16);
      *reinterpret_cast<uint4 *>(xq + 4) = *reinterpret_cast<const uint4 *>(tq + r * LD + kc * 16 + 8);
      *reinterpret_cast<uint4 *>(xk) = *reinterpret_cast<const uint4 *>(tk + r * LD + kc * 16);
      *reinterpret_cast<uint4 *>(xk + 4) = *reinterpret_cast<const uint4 *>(tk + r * LD + kc * 16 + 8);
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const float fq = __uint_as_float((i & 1) ? (xq[i >> 1] & 0xffff0000u) : (xq[i >> 1] << 16));
        const float fk = __uint_as_float((i & 1) ? (xk[i >> 1] & 0xffff0000u) : (xk[i >> 1] << 16));
        const int cq = round_half_away(dq.fast ? dq.quick(fq) : dq.exact(fq));
        const int ck = round_half_away(dk.fast ? dk.quick(fk) : dk.exact(fk));
        wq[i >> 2] |= (uint32_t)(cq & 0xff) << (8 * (i & 3));
        wk[i >> 2] |= (uint32_t)(ck & 0xff) << (8 * (i & 3));
      }
      *reinterpret_cast<uint4 *>(qr + (size_t)idx * 16) = make_uint4(wq[0], wq[1], wq[2], wq[3]);
      *reinterpret_cast<uint4 *>(kr + (size_t)idx * 16) = make_uint4(wk[0], wk[1], wk[2], wk[3]);
    }
    for (int idx = tid; idx < D * kSlots / 16; idx += NT) {  // chunk (kc, c): slots kc*16.. of channel c
      const int kc = idx / D, c = idx % D;
      const float dv = p.dv8[(size_t)bh * D + c];
      uint32_t w[4] = {0, 0, 0, 0};
      if (dv > 0.f) {
        const Divider div = make_divider(dv);
        const uint32_t m16 = (uint32_t)(mask >> (kc * 16)) & 0xffffu;
        if (div.fast) {
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const uint32_t code = cast_e4m3(div.quick(bf16_to_f32(tv[(kc * 16 + i) * LD + c])));
            w[i >> 2] |= ((m16 >> i) & 1u) ? code << (8 * (i & 3)) : 0u;
          }
        } else {
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const uint32_t code = cast_e4m3(div.exact(bf16_to_f32(tv[(kc * 16 + i) * LD + c])));
            w[i >> 2] |= ((m16 >> i) & 1u) ? code << (8 * (i & 3)) : 0u;
          }
        }
      }
      *reinterpret_cast<uint4 *>(vr + (size_t)idx * 16) = make_uint4(w[0], w[1], w[2], w[3]);
    }
  }

  // ------------------------------------------------------------------ tier 0: NVFP4
  if (p.tier_active[0] && video) {
    const float gq = p.gscale[bh * 4 + 0], gk = p.gscale[bh * 4 + 1], gv = p.gscale[bh * 4 + 2];
    constexpr int QK_IMG = kSlots * D / 2, NATOM = D / 64;
    uint8_t *qr = p.qrec[0] + blk * p.qrec_bytes[0];
    uint8_t *kr = p.kvrec[0] + blk * p.kvrec_bytes[0];
    uint8_t *vr = kr + QK_IMG + NATOM * kSfAtomBytes;
    for (int which = 0; which < 2; ++which) {  // 0: Q, 1: K
      const uint16_t *src = which ? tk : tq;
      uint8_t *dst = which ? kr : qr;
      const float g = which ? gk : gq;
      __syncthreads();
      for (int i = tid; i < NATOM * kSfAtomBytes / 4; i += NT) reinterpret_cast<uint32_t *>(sf_img)[i] = 0;
      __syncthreads();
      for (int idx = tid; idx < kSlots * D / 32; idx += NT) {  // chunk (kc, r): channels kc*32.. of slot r
        const int kc = idx / kSlots, r = idx % kSlots;
        uint32_t w[4];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          float x[16];
          uint32_t pk[2];
#pragma unroll
          for (int i = 0; i < 16; ++i) x[i] = bf16_to_f32(src[r * LD + kc * 32 + h * 16 + i]);
          const uint32_t sc = nvfp4_group(x, g, pk);
          w[2 * h] = pk[0]; w[2 * h + 1] = pk[1];
          const int grp = kc * 2 + h;  // 16-channel group index; 4 groups per atom
          // rows 0..63 and, duplicated, rows 64..127: the attention kernel places a block's queries in either half
          uint8_t *sfp = sf_img + (grp >> 2) * kSfAtomBytes + (r & 31) * 16 + (r >> 5) * 4 + (grp & 3);
          sfp[0] = (uint8_t)sc;
          sfp[8] = (uint8_t)sc;
        }
        *reinterpret_cast<uint4 *>(dst + (size_t)idx * 16) = make_uint4(w[0], w[1], w[2], w[3]);
      }
      __syncthreads();
      for (int i = tid; i < NATOM * kSfAtomBytes / 16; i += NT)
        *reinterpret_cast<uint4 *>(dst + QK_IMG + (size_t)i * 16) = reinterpret_cast<const uint4 *>(sf_img)[i];
    }
    __syncthreads();
    for (int i = tid; i < kSfAtomBytes / 4; i += NT) reinterpret_cast<uint32_t *>(sf_img)[i] = 0;
    __syncthreads();
    for (int idx = tid; idx < D * kSlots / 32; idx += NT) {  // chunk (kc, c): slots kc*32.. of channel c
      const int kc = idx / D, c = idx % D;
      uint32_t w[4];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        float x[16];
        uint32_t pk[2];
#pragma unroll
        for (int i = 0; i < 16; ++i) x[i] = bf16_to_f32(tv[(kc * 32 + h * 16 + i) * LD + c]);
        const uint32_t sc = nvfp4_group(x, gv, pk);
        w[2 * h] = pk[0]; w[2 * h + 1] = pk[1];
        sf_img[(c & 31) * 16 + (c >> 5) * 4 + (kc * 2 + h)] = (uint8_t)sc;
      }
      *reinterpret_cast<uint4 *>(vr + (size_t)idx * 16) = make_uint4(w[0], w[1], w[2], w[3]);
    }
    __syncthreads();
    for (int i = tid; i < kSfAtomBytes / 16; i += NT)
      *reinterpret_cast<uint4 *>(vr + D * kSlots / 2 + (size_t)i * 16) = reinterpret_cast<const uint4 *>(sf_img)[i];
  }
}

// Self-check of Divider::quick and round_half_away against the IEEE division and roundf (see da2.h).
__device__ __forceinline__ uint32_t mix32(uint32_t x) {
  x ^= x >> 16; x *= 0x7feb352dU; x ^= x >> 15; x *= 0x846ca68bU; x ^= x >> 16;
  return x;
}
__global__ void selfcheck_quotient_kernel(int n_divisors, int all_ones, uint32_t seed, unsigned long long *bad_out) {
  const int di = blockIdx.x * blockDim.x + threadIdx.x;
  if (di >= n_divisors) return;
  const uint32_t h = mix32((uint32_t)di * 2654435761u + seed);
  const uint32_t man = all_ones ? 0x7fffffu : (h & 0x7fffffu);
  const uint32_t ex = 127u - 60u + mix32(h) % 120u;  // binades 2^-60 .. 2^59: inside the quick range
  const Divider div = make_divider(__uint_as_float((ex << 23) | man));
  unsigned long long bad = div.fast ? 0ull : 1ull;
  for (uint32_t b = 0; b < 65536u; ++b) {
    const float x = __uint_as_float(b << 16);
    if (!(fabsf(x) <= 3.0e38f) || (x != 0.f && fabsf(x) < 7.9e-31f)) continue;  // finite, zero or at least 2^-100
    const float ref = div.exact(x);
    if (!(fabsf(ref) < 3.0e38f) || (ref != 0.f && fabsf(ref) < 1e-30f)) continue;  // quotient in the normal range
    if (__float_as_uint(div.quick(x)) != __float_as_uint(ref)) ++bad;
  }
  if (bad) atomicAdd(bad_out, bad);
}
__global__ void selfcheck_round_kernel(unsigned long long *bad_out) {
  const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
  unsigned long long bad = 0;
  for (unsigned long long b = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; b < (1ull << 32); b += stride) {
    const float x = __uint_as_float((uint32_t)b);
    if (!(fabsf(x) < 8388608.0f)) continue;
    if ((int)roundf(x) != round_half_away(x)) ++bad;
  }
  if (bad) atomicAdd(bad_out, bad);
}

}  // namespace

cudaError_t launch_quantiser_selfcheck(int mode, int n_divisors, uint32_t seed, unsigned long long *out, cudaStream_t st) {
  cudaError_t e = cudaMemsetAsync(out, 0, sizeof(unsigned long long), st);
  if (e != cudaSuccess) return e;
  if (mode == 2) selfcheck_round_kernel<<<148 * 8, 256, 0, st>>>(out);
  else selfcheck_quotient_kernel<<<(n_divisors + 127) / 128, 128, 0, st>>>(n_divisors, mode == 1, seed, out);
  return cudaGetLastError();
}

cudaError_t launch_prep(const Params &p, const __nv_bfloat16 *q, const __nv_bfloat16 *k, const __nv_bfloat16 *v,
                        cudaStream_t st, int *launches, bool pool) {
  dim3 grid(p.Rt, p.BH);
  const size_t smem = 3 * (size_t)kSlots * (p.d + 8) * 2 + 3 * kSfAtomBytes;
  auto launch = [&](auto kernel) -> cudaError_t {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kernel<<<grid, NT, smem, st>>>(p, q, k, v);
    return cudaGetLastError();
  };
  cudaError_t e;
  if (p.d == 128) e = pool ? launch(prep_kernel<128, true>) : launch(prep_kernel<128, false>);
  else e = pool ? launch(prep_kernel<64, true>) : launch(prep_kernel<64, false>);
  if (e != cudaSuccess) return e;
  *launches += 1;
  return cudaSuccess;
}

}  // namespace da2
