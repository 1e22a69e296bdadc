// Kernel 4: phased mixed-precision block-sparse attention (Sec. 3.3 "Phased execution" and "Cross-precision
// accumulation", App. C.3 / C.4).
//
// One CTA owns one query block (64 tokens) and walks its list: NVFP4 segment, then INT8/E4M3 segment, then BF16
// segment.  All segments share the fp32 running row maximum h, the fp32 denominator l (which always sums the
// exponential weights BEFORE they are converted to a matrix operand) and ONE output accumulator in tensor memory;
// at a segment boundary the accumulator only changes units (Eq. "precision-state-conversion"), and the output is
// normalised once at the end.
//
// Mapping onto sm_100a:
//   S   = Q K^T   : tcgen05.mma, M = 128 (rows 0..63 are the block's queries, rows 64..127 are don't-care rows the
//                   block-scaled instruction shape requires), N = 64 keys, K = d; fp32 / int32 accumulator in TMEM.
//   O^T = V^T P^T : tcgen05.mma, M = 128 (channels; d = 64 leaves rows 64..127 unused), N = 64 queries, K = 64 keys.
//                   Keeping O transposed makes the online-softmax correction a per-COLUMN scale, so only the queries
//                   whose maximum moved are touched, and makes the per-channel unit changes a per-lane scalar.
//   kinds         : kind::f16 (BF16), kind::i8 for QK^T + kind::f8f6f4 (E4M3 x E4M3) for PV (App. C.1: the INT8 path
//                   uses INT8 for QK^T and FP8 for PV), kind::mxf4nvf4 with E4M3 scales per 16 elements (NVFP4).
//   operands      : da2_prepare wrote every block as a ready shared-memory image, so one 1-D bulk copy per step
//                   brings K, V^T and their scale factors; P and its NVFP4 scale factors are produced by the softmax
//                   threads into shared memory (tcgen05.cp moves scale factors into TMEM).
// Every wait on an mbarrier is bounded; a wait that gives up records DA2 device status "timeout" and the CTA winds
// down normally (TMEM released).
#include <cuda_fp8.h>

#include "da2_internal.cuh"
#include "tc05.cuh"

namespace da2 {

namespace {

constexpr int NT = 128;
constexpr uint32_t kTmemCols = 256;
constexpr uint32_t COL_S = 0, COL_O = 64, COL_SFQ = 128, COL_SFK = 136, COL_SFV = 144, COL_SFP = 148;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kEtaP8 = 0.0022326917f;  // probability dequantisation scale of the 8-bit path
constexpr float kOffsetP8 = 8.807f;      // base-2 exponent offset (about log2 448)

struct SmemMap {
  uint32_t q[3];     // Q record per tier (only active tiers are resident)
  uint32_t kv[2];    // two K/V stages
  uint32_t p;        // P operand image, 64 x 64 x <= 2 bytes
  uint32_t sfp;      // P scale atom (512 B)
  uint32_t factor;   // 64 floats: per-query correction factor of this step
  uint32_t inv_l;    // 64 floats
  uint32_t changed;  // 64 bytes: 1 if the query's maximum moved this step
  uint32_t bars;     // mbarriers
  uint32_t total;
  uint32_t kv_bytes;
};

__host__ SmemMap make_smem_map(const Params &p) {
  SmemMap m;
  uint32_t cur = 0;
  auto take = [&](uint32_t bytes) { uint32_t o = cur; cur = (cur + bytes + 127u) / 128u * 128u; return o; };
  for (int t = 0; t < 3; ++t) m.q[t] = p.tier_active[t] ? take(p.qrec_bytes[t]) : 0;
  uint32_t kvb = 0;
  for (int t = 0; t < 3; ++t)
    if (p.tier_active[t] && p.kvrec_bytes[t] > kvb) kvb = p.kvrec_bytes[t];
  if (kvb < 16384) kvb = 16384;  // stage 0 doubles as the output staging tile [64][d] bf16
  m.kv_bytes = kvb;
  m.kv[0] = take(kvb);
  m.kv[1] = take(kvb);
  m.p = take(8192);
  m.sfp = take(512);
  m.factor = take(256);
  m.inv_l = take(256);
  m.changed = take(64);
  m.bars = take(64);
  m.total = cur;
  return m;
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ uint32_t pack_e4m3x2(float lo, float hi) {
  uint16_t r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
  return (uint32_t)r;
}
__device__ __forceinline__ uint32_t pack_e2m1x2(float lo, float hi) {
  uint16_t r;
  asm("{ .reg .b8 t; cvt.rn.satfinite.e2m1x2.f32 t, %2, %1; mov.b16 %0, {t, 0}; }" : "=h"(r) : "f"(lo), "f"(hi));
  return (uint32_t)r;
}
__device__ __forceinline__ float decode_e4m3(uint32_t c) {
  const __half_raw h = __nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)c, __NV_E4M3);
  return __half2float(*reinterpret_cast<const __half *>(&h));
}

// bounded wait that also gives up as soon as another thread of the CTA has flagged a failure
__device__ __forceinline__ bool wait_or_abort(uint64_t *bar, uint32_t parity, volatile int *abort_flag) {
  for (uint32_t i = 0; i < (1u << 22); ++i) {
    if (tc::mbar_try_wait(bar, parity)) return true;
    if (i > 32) {
      __nanosleep(128);
      if (*abort_flag) return false;
    }
  }
  return false;
}

template <int D>
__global__ void __launch_bounds__(NT) attention_kernel(Params p, SmemMap sm, __nv_bfloat16 *__restrict__ out) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_abort;

  const int tid = threadIdx.x, warp = tid >> 5;
  const int bh = blockIdx.x / p.R, a = blockIdx.x % p.R;
  const int R = p.R;
  const int *cnt = p.counts + ((size_t)bh * R + a) * 4;
  const int n4 = cnt[0], n8 = cnt[1], n16 = cnt[2];
  const int L = n4 + n8 + n16;
  const uint16_t *ids = p.ids + (size_t)bh * p.ids_per_head + cnt[3];
  const unsigned long long qmask = block_valid_mask(p, a);
  __nv_bfloat16 *out_head = out + (size_t)bh * p.N * D;

  if (L == 0) {  // no retained key: the rows return zero (App. C.1)
    for (int idx = tid; idx < kSlots * (D / 8); idx += NT) {
      const int j = idx / (D / 8), c8 = idx % (D / 8);
      if ((qmask >> j) & 1ull)
        *reinterpret_cast<uint4 *>(out_head + (size_t)slot_token(p, a, j) * D + c8 * 8) = make_uint4(0, 0, 0, 0);
    }
    return;
  }

  uint64_t *bars = reinterpret_cast<uint64_t *>(smem + sm.bars);
  uint64_t *bar_full = bars;      // [2]
  uint64_t *bar_q = bars + 2;
  uint64_t *bar_s = bars + 3;
  uint64_t *bar_o = bars + 4;
  float *s_factor = reinterpret_cast<float *>(smem + sm.factor);
  float *s_inv_l = reinterpret_cast<float *>(smem + sm.inv_l);
  uint8_t *s_changed = smem + sm.changed;

  if (warp == 0) {
    tc::tmem_alloc(&s_tmem_base, kTmemCols);
    tc::tmem_relinquish();
  }
  if (tid == 0) {
    tc::mbar_init(&bar_full[0], 1);
    tc::mbar_init(&bar_full[1], 1);
    tc::mbar_init(bar_q, 1);
    tc::mbar_init(bar_s, 1);
    tc::mbar_init(bar_o, 1);
    tc::fence_barrier_init();
    s_abort = 0;
  }
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tmem = s_tmem_base;

  auto tier_of_step = [&](int i) { return i < n4 ? 0 : (i < n4 + n8 ? 1 : 2); };
  auto issue_kv = [&](int i) {  // thread 0 only
    const int t = tier_of_step(i);
    int b = ids[i];
    if (b >= R) { atomicExch(p.status, kDevBadList); b = 0; }
    const uint8_t *src = p.kvrec[t] + ((size_t)bh * R + b) * p.kvrec_bytes[t];
    tc::mbar_arrive_expect_tx(&bar_full[i & 1], p.kvrec_bytes[t]);
    tc::bulk_g2s(smem + sm.kv[i & 1], src, p.kvrec_bytes[t], &bar_full[i & 1]);
  };

  if (tid == 0) {
    uint32_t qbytes = 0;
    const int nn[3] = {n4, n8, n16};
    for (int t = 0; t < 3; ++t) if (nn[t] > 0) qbytes += p.qrec_bytes[t];
    tc::mbar_arrive_expect_tx(bar_q, qbytes);
    for (int t = 0; t < 3; ++t)
      if (nn[t] > 0)
        tc::bulk_g2s(smem + sm.q[t], p.qrec[t] + ((size_t)bh * R + a) * p.qrec_bytes[t], p.qrec_bytes[t], bar_q);
    issue_kv(0);
    if (L > 1) issue_kv(1);
  }

  // per-row online-softmax state (threads 0..63 own query rows; log2 domain)
  float h2 = -INFINITY, ell = 0.f;
  const float gq = p.gscale[bh * 4 + 0], gk = p.gscale[bh * 4 + 1], gv = p.gscale[bh * 4 + 2];
  const float dq8 = p.tier_active[1] ? p.dq8[(size_t)bh * R + a] : 0.f;
  const float dv8 = (p.tier_active[1] && tid < D) ? p.dv8[(size_t)bh * D + tid] : 0.f;
  const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
  auto unit_of = [&](int t) -> float {  // common units per accumulator unit, for this thread's channel
    return t == 0 ? __fdiv_rn(gv, 2688.0f) : (t == 1 ? kEtaP8 * dv8 : 1.0f);
  };
  int prev_tier = -1;
  bool failed = false;

  if (!wait_or_abort(bar_q, 0, &s_abort)) { s_abort = 1; failed = true; }
  if (tid == 0 && n4 > 0 && !failed) {  // Q scale factors go to TMEM once
    for (int i = 0; i < D / 64; ++i)
      tc::tmem_cp_sf(tmem + COL_SFQ + 4 * i,
                     tc::smem_desc(tc::smem_u32(smem + sm.q[0] + kSlots * D / 2 + i * kSfAtomBytes), 128, 128));
  }
  __syncthreads();

  for (int i = 0; i < L && !s_abort; ++i) {
    const int tier = tier_of_step(i);
    const int b = min((int)ids[i], R - 1);
    const uint32_t kvs = tc::smem_u32(smem + sm.kv[i & 1]);

    // ------------------------------------------------------------ S = Q K^T (one thread issues)
    if (tid == 0) {
      if (!wait_or_abort(&bar_full[i & 1], (i >> 1) & 1, &s_abort)) { s_abort = 1; }
      else {
        tc::fence_after_sync();
        const uint32_t qs = tc::smem_u32(smem + sm.q[tier]);
        if (tier == 2) {
          for (int ks = 0; ks < D / 16; ++ks)
            tc::mma_f16(tmem + COL_S, tc::smem_desc(qs + ks * 2048, 1024, 128),
                        tc::smem_desc(kvs + ks * 2048, 1024, 128), tc::idesc_bf16(64), ks > 0);
        } else if (tier == 1) {
          for (int ks = 0; ks < D / 32; ++ks)
            tc::mma_i8(tmem + COL_S, tc::smem_desc(qs + ks * 2048, 1024, 128),
                       tc::smem_desc(kvs + ks * 2048, 1024, 128), tc::idesc_i8(64), ks > 0);
        } else {
          const uint32_t ksf = kvs + kSlots * D / 2;
          for (int j = 0; j < D / 64; ++j)
            tc::tmem_cp_sf(tmem + COL_SFK + 4 * j, tc::smem_desc(ksf + j * kSfAtomBytes, 128, 128));
          const uint32_t vsf = ksf + (D / 64) * kSfAtomBytes + D * kSlots / 2;
          tc::tmem_cp_sf(tmem + COL_SFV, tc::smem_desc(vsf, 128, 128));
          for (int ks = 0; ks < D / 64; ++ks)
            tc::mma_nvfp4(tmem + COL_S, tc::smem_desc(qs + ks * 2048, 1024, 128),
                          tc::smem_desc(kvs + ks * 2048, 1024, 128), tc::idesc_nvfp4(64), ks > 0,
                          tmem + COL_SFQ + 4 * ks, tmem + COL_SFK + 4 * ks);
        }
        tc::mma_commit(bar_s);
      }
    }
    if (!wait_or_abort(bar_s, i & 1, &s_abort)) { s_abort = 1; }
    tc::fence_after_sync();

    // ------------------------------------------------------------ online softmax, one thread per query row
    if (tid < kSlots && !s_abort) {
      uint32_t raw[64];
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t part[16];
        tc::tmem_ld16(tmem + lane_base + COL_S + 16 * c, part);
#pragma unroll
        for (int j = 0; j < 16; ++j) raw[16 * c + j] = part[j];
      }
      tc::wait_ld();
      const unsigned long long kmask = block_valid_mask(p, b);
      float coef;
      if (tier == 2) coef = p.scale * kLog2e;
      else if (tier == 1) coef = dq8 * p.dk8[(size_t)bh * R + b] * p.scale * kLog2e;
      else coef = gq * gk * p.scale * kLog2e;
      float t[64];
      float mloc = -INFINITY;
#pragma unroll
      for (int j = 0; j < 64; ++j) {
        const float sv = tier == 1 ? (float)(int)raw[j] : __uint_as_float(raw[j]);
        t[j] = ((kmask >> j) & 1ull) ? sv * coef : -INFINITY;
        mloc = fmaxf(mloc, t[j]);
      }
      const float m_new = fmaxf(h2, mloc);
      const float factor = ex2(h2 - m_new);  // 0 on the first block (h2 = -inf)
      s_factor[tid] = factor;
      s_changed[tid] = (m_new != h2) ? 1 : 0;
      ell *= factor;
      h2 = m_new;
      uint8_t *prow = smem + sm.p + tid * 16;
      if (tier == 2) {
        float sum = 0.f;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          uint32_t w4[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const float w0 = ex2(t[c * 8 + 2 * j] - m_new), w1 = ex2(t[c * 8 + 2 * j + 1] - m_new);
            sum += w0 + w1;
            w4[j] = pack_bf16x2(w0, w1);
          }
          *reinterpret_cast<uint4 *>(prow + c * 1024) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
        }
        ell += sum;
      } else if (tier == 1) {
        float sum = 0.f;
        const float shift = kOffsetP8 - m_new;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t w4[4] = {0, 0, 0, 0};
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float w0 = ex2(t[c * 16 + 2 * j] + shift), w1 = ex2(t[c * 16 + 2 * j + 1] + shift);
            sum += w0 + w1;
            w4[j >> 1] |= pack_e4m3x2(w0, w1) << (16 * (j & 1));
          }
          *reinterpret_cast<uint4 *>(prow + c * 1024) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
        }
        ell += kEtaP8 * sum;  // the denominator accumulates the amplified fp32 weights; eta restores the unit
      } else {
        float sum = 0.f;
        uint32_t sfword = 0;
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          float w[16];
          float gm = 0.f;
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            w[j] = ex2(t[g * 16 + j] - m_new);
            sum += w[j];
            gm = fmaxf(gm, w[j]);
          }
          const uint32_t sc = pack_e4m3x2(__fmul_rn(448.0f, gm), 0.f) & 0xffu;
          const float sigma = decode_e4m3(sc);
          sfword |= sc << (8 * g);
          uint32_t w2[2] = {0, 0};
          if (sigma > 0.f) {
            const float inv = __fdiv_rn(2688.0f, sigma);
#pragma unroll
            for (int j = 0; j < 8; ++j) w2[j >> 2] |= pack_e2m1x2(w[2 * j] * inv, w[2 * j + 1] * inv) << (8 * (j & 3));
          }
          // 16 keys = 8 bytes: chunk g/2 (32 keys per 16-byte chunk), half g&1
          *reinterpret_cast<uint2 *>(prow + (g >> 1) * 1024 + (g & 1) * 8) = make_uint2(w2[0], w2[1]);
        }
        *reinterpret_cast<uint32_t *>(smem + sm.sfp + (tid & 31) * 16 + (tid >> 5) * 4) = sfword;
        ell += sum;
      }
      tc::fence_async_smem();
    }
    tc::fence_before_sync();
    __syncthreads();
    tc::fence_after_sync();
    if (s_abort) break;

    // ------------------------------------------------------------ correct the accumulator (all 128 lanes)
    if (i > 0) {
      float lane_factor = 1.0f;
      const bool tier_switch = tier != prev_tier;
      if (tier_switch && tid < D) {
        const float un = unit_of(tier), up = unit_of(prev_tier);
        lane_factor = un > 0.f ? __fdiv_rn(up, un) : 0.f;
      }
#pragma unroll 1
      for (int c = 0; c < 8; ++c) {
        const unsigned long long ch = *reinterpret_cast<const unsigned long long *>(s_changed + c * 8);
        if (ch == 0ull && !tier_switch) continue;
        uint32_t o[8];
        tc::tmem_ld8(tmem + lane_base + COL_O + c * 8, o);
        tc::wait_ld();
#pragma unroll
        for (int j = 0; j < 8; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * (s_factor[c * 8 + j] * lane_factor));
        tc::tmem_st8(tmem + lane_base + COL_O + c * 8, o);
      }
      tc::wait_st();
    }
    prev_tier = tier;
    tc::fence_before_sync();
    __syncthreads();

    // ------------------------------------------------------------ O^T += V^T P^T (one thread issues)
    if (tid == 0) {
      tc::fence_after_sync();
      const uint32_t ps = tc::smem_u32(smem + sm.p);
      if (tier == 2) {
        const uint32_t vs = kvs + kSlots * D * 2;
        for (int ks = 0; ks < 4; ++ks)
          tc::mma_f16(tmem + COL_O, tc::smem_desc(vs + ks * 2 * D * 16, D * 16, 128),
                      tc::smem_desc(ps + ks * 2048, 1024, 128), tc::idesc_bf16(64), (i > 0) || (ks > 0));
      } else if (tier == 1) {
        const uint32_t vs = kvs + kSlots * D;
        for (int ks = 0; ks < 2; ++ks)
          tc::mma_f8f6f4(tmem + COL_O, tc::smem_desc(vs + ks * 2 * D * 16, D * 16, 128),
                         tc::smem_desc(ps + ks * 2048, 1024, 128), tc::idesc_e4m3(64), (i > 0) || (ks > 0));
      } else {
        const uint32_t vs = kvs + kSlots * D / 2 + (D / 64) * kSfAtomBytes;
        tc::tmem_cp_sf(tmem + COL_SFP, tc::smem_desc(tc::smem_u32(smem + sm.sfp), 128, 128));
        tc::mma_nvfp4(tmem + COL_O, tc::smem_desc(vs, D * 16, 128), tc::smem_desc(ps, 1024, 128),
                      tc::idesc_nvfp4(64), i > 0, tmem + COL_SFV, tmem + COL_SFP);
      }
      tc::mma_commit(bar_o);
    }
    if (!wait_or_abort(bar_o, i & 1, &s_abort)) { s_abort = 1; }
    tc::fence_after_sync();
    __syncthreads();
    if (tid == 0 && i + 2 < L && !s_abort) issue_kv(i + 2);
  }

  if (s_abort) {
    if (tid == 0) {
      atomicExch(p.status, kDevTimeout);
      // let any copy still in flight land before the shared memory goes away
      tc::mbar_wait(&bar_full[0], 0, 1u << 16);
      tc::mbar_wait(&bar_full[1], 0, 1u << 16);
    }
  } else {
    // ---------------------------------------------------------- epilogue: O = U / l, back to raster order
    if (tid < kSlots) s_inv_l[tid] = ell > 0.f ? __fdiv_rn(1.0f, ell) : 0.f;
    __syncthreads();
    uint16_t *stage = reinterpret_cast<uint16_t *>(smem + sm.kv[0]);  // [64][D] bf16
    const float unit = tid < D ? unit_of(prev_tier) : 0.f;
#pragma unroll 1
    for (int c = 0; c < 8; ++c) {
      uint32_t o[8];
      tc::tmem_ld8(tmem + lane_base + COL_O + c * 8, o);
      tc::wait_ld();
      if (tid < D) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const float val = __uint_as_float(o[j]) * unit * s_inv_l[c * 8 + j];
          stage[(c * 8 + j) * D + tid] = __bfloat16_as_ushort(__float2bfloat16_rn(val));
        }
      }
    }
    __syncthreads();
    for (int idx = tid; idx < kSlots * (D / 8); idx += NT) {
      const int j = idx / (D / 8), c8 = idx % (D / 8);
      if ((qmask >> j) & 1ull)
        *reinterpret_cast<uint4 *>(out_head + (size_t)slot_token(p, a, j) * D + c8 * 8) =
            *reinterpret_cast<const uint4 *>(stage + j * D + c8 * 8);
    }
  }
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 0) tc::tmem_dealloc(tmem, kTmemCols);
}

}  // namespace

cudaError_t launch_attention(const Params &p, __nv_bfloat16 *out, cudaStream_t st, int *launches) {
  const SmemMap sm = make_smem_map(p);
  cudaError_t e;
  const int grid = p.BH * p.R;
  if (p.d == 128) {
    e = cudaFuncSetAttribute(attention_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm.total);
    if (e != cudaSuccess) return e;
    attention_kernel<128><<<grid, NT, sm.total, st>>>(p, sm, out);
  } else {
    e = cudaFuncSetAttribute(attention_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm.total);
    if (e != cudaSuccess) return e;
    attention_kernel<64><<<grid, NT, sm.total, st>>>(p, sm, out);
  }
  *launches += 1;
  return cudaGetLastError();
}

}  // namespace da2
