// Kernel 4: phased mixed-precision block-sparse attention (Sec. 3.3 "Phased execution" and "Cross-precision
// accumulation", App. C.3 / C.4).
//
// Every query block (64 tokens) walks its own list: NVFP4 segment, then INT8/E4M3 segment, then BF16 segment.  All
// segments share the fp32 running row maximum h, the fp32 denominator l (which always sums the exponential weights
// BEFORE they are converted to a matrix operand) and ONE output accumulator in tensor memory; at a segment boundary
// the accumulator only changes units (Eq. "precision-state-conversion"), and the output is normalised once.
//
// Mapping onto sm_100a
//   A CTA owns two neighbouring query blocks ("streams" 0 and 1) and 1024 threads (768 when shared memory only
//   leaves room for two softmax sets) in six roles, with S = 4 (or 2) softmax sets:
//     warps 0..4S-1   softmax, set k = warp/4 takes the steps i = k (mod S); inside a set stream = (warp%4)/2 and one
//                     thread owns one full 64-key row.  A thread reads its S row from TMEM, takes the running maximum
//                     of step i-1 from the thread of the previous set through a shared-memory word tagged with the
//                     step, keeps a partial denominator, and writes P~ (and its NVFP4 scale factors) into its set's
//                     operand image.  These warps hold most of the register file (setmaxnreg).
//     next 8 warps    correction + epilogue, four per stream.  Every step passes through them between the softmax
//                     and the product: they read the step's "maximum moved" ballots and, only if one is set or the
//                     segment changes, wait for the previous product and rescale those accumulator columns (and apply
//                     the per-channel unit change); then they release the product.  Most steps move no maximum, and
//                     the check is off the issuing warp's instruction stream.  Finally they combine the sets' partial
//                     denominators, normalise, transpose and store
//     next 2 warps    S = Q K^T issue, one warp per stream (tcgen05.mma, accumulators in TMEM), two steps ahead
//     next 2 warps    O^T += V^T P~^T issue, one warp per stream.  The issuing warps' instruction
//                     counts are on the critical path of every step: their loops are warp-uniform (one elected lane
//                     issues), operand descriptors are built once and only offset inside the loop
//     last 4 warps    loaders: per stream one warp for K (and the Q records) and one for V^T, 1-D bulk copies into
//                     rings of their own (a K block is needed as soon as a score buffer is free, a V block only after
//                     the step's weights are written, so the V ring is the deeper one); lane l holds list entry
//                     32*batch + l (address, mask, key scale)
//   S   = Q K^T   : M = 128, N = 64 keys, K = d.  The block-scaled instruction only exists at M = 128, so stream 0's
//                   queries sit in rows 0..63 and stream 1's in rows 64..127 (its operand descriptor starts 1 KB
//                   early); the other 64 rows of each product are don't-care.  S is double buffered.
//   O^T = V^T P^T : M = 128 channels, N = 64 queries, K = 64 keys.  Keeping O transposed makes the online-softmax
//                   correction a per-COLUMN scale, so only queries whose maximum moved are touched, and makes the
//                   per-channel unit changes (eta*delta_c^V, g_V/2688) per-lane scalars.
//   kinds         : kind::f16 (BF16); kind::i8 for QK^T + kind::f8f6f4 E4M3 x E4M3 for PV (App. C.1); and
//                   kind::mxf4nvf4 with E4M3 scales per 16 elements (NVFP4), scale factors moved by tcgen05.cp.
// The softmax sets the pace (per score: one ex2 on a 16-lane/clk unit plus the quantisation arithmetic): the row
// maximum is taken on raw accumulator values, the scale and the maximum are folded into one FMA feeding ex2, int32
// scores become floats through a magic-number add, the NVFP4 group scale is folded into the exponent so the scaled
// weight needs no extra multiply, and the exponentiate phase runs over the whole row in batches (all arguments, all
// exponentials, then sums and packing), which gives the single warp the instruction-level parallelism it lacks when
// the three are interleaved per pair.
// Every wait on an mbarrier is bounded; a wait that gives up records device status "timeout", all roles leave their
// loops and the CTA exits normally after releasing TMEM.
#include <type_traits>
#include <cuda_fp8.h>

#include "da2_internal.cuh"
#include "tc05.cuh"

namespace da2 {

namespace {

// Softmax warp sets: set k takes the steps i = k (mod SETS), one thread per 64-key row, four warps (one per TMEM lane
// quarter) per set.  Plans without a 16-bit tier run four sets; a 16-bit tier needs 8 KB per P image and 16 KB ring
// stages, which leaves shared memory for two.
constexpr int kMaxSets = 4;
template <int SETS> struct Roles {
  static constexpr int kSoftmaxWarps = 4 * SETS, kCorrWarps = 8;  // four correction warps per stream
  static constexpr int kMmaWarp0 = kSoftmaxWarps + kCorrWarps;    // Q K^T issue for stream 0, 1
  static constexpr int kPvWarp0 = kMmaWarp0 + 2;                  // V^T P^T issue for stream 0, 1
  static constexpr int kLoadWarp0 = kPvWarp0 + 2;                 // K loaders for stream 0, 1, then V loaders
  static constexpr int NT = (kLoadWarp0 + 4) * 32;                // 1024 (four sets) or 768 (two): whole warpgroups
  static constexpr int kShift = SETS == 4 ? 2 : 1, kMask = SETS - 1;
};
constexpr uint32_t kTmemCols = 512;
// TMEM column map
__host__ __device__ constexpr uint32_t col_s(int s, int buf) { return (uint32_t)(s * 2 + buf) * 64u; }
__host__ __device__ constexpr uint32_t col_o(int s) { return 256u + (uint32_t)s * 64u; }
// scale factors: every region starts on a multiple of 4 columns (one 4-column group holds 128 rows x 4 scales)
__host__ __device__ constexpr uint32_t col_sfq(int s) { return 384u + (uint32_t)s * 8u; }  // 4 columns per K step
__host__ __device__ constexpr uint32_t col_sfk(int s) { return 400u + (uint32_t)s * 8u; }
__host__ __device__ constexpr uint32_t col_sfv(int s) { return 416u + (uint32_t)s * 4u; }
__host__ __device__ constexpr uint32_t col_sfp(int s) { return 424u + (uint32_t)s * 4u; }

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kEtaP8 = 0.0022326917f;  // probability dequantisation scale of the 8-bit path
constexpr float kOffsetP8 = 8.807f;      // base-2 exponent offset (about log2 448)

// barrier indices inside one stream's group
// (a parity wait can only tell the latest completion from the one before, so every barrier is laid out such that no
// waiter can fall two completions behind: buffers indexed by step parity get one barrier per buffer)
enum { B_FULLK = 0, B_FULLV = 4, B_KFREE = 10, B_VFREE = 14, B_SREADY = 20, B_SFREE = 24, B_PREADY = 26, B_CORROK = 30, B_PVDONE = 34, B_ELL = 38, B_Q = 39, B_COUNT = 40 };
constexpr int kMaxK = 4, kMaxV = 6, kInfoRing = 8;

struct SmemMap {
  uint32_t q[2][3];   // Q record per stream and tier
  uint32_t kst[2][kMaxK];  // K ring per stream (K image + its scale atoms)
  uint32_t vst[2][kMaxV];  // V ring per stream (V^T image + its scale atom)
  int nk, nv;                   // ring depths
  uint32_t kbytes[3], vbytes[3];
  uint32_t p[2][kMaxSets];   // P operand images per stream, one per softmax set (64 x 64 x <= 2 bytes)
  uint32_t sfp[2][kMaxSets]; // P scale atoms (512 B)
  uint32_t factor;    // float [2 streams][sets][64]
  uint32_t hx;        // {float h, int step} [2][sets][64]: running maximum after a step, handed from thread to thread
  uint32_t href;      // float [2][sets][64]: reference of each set's partial denominator
  uint32_t ell;       // float [2][sets][64]
  uint32_t info;      // per stream, ring of kInfoRing steps: {u64 mask, float dk8, pad}
  uint32_t bars;      // uint64 [2][B_COUNT]
  uint32_t kstage, vstage;  // bytes per ring stage
  uint32_t pbytes;          // bytes of one P image (the kSets images of a stream are contiguous)
  uint32_t chg;             // uint32 [2 streams][sets][2]: ballots of the queries whose maximum moved this step
  uint32_t total;
  bool fits;                // the layout fits the 227 KB a block may use
};

__host__ SmemMap make_smem_map(const Params &p, int kSets) {
  SmemMap m;
  uint32_t cur = 0;
  auto take = [&](uint32_t bytes) { uint32_t o = cur; cur = (cur + bytes + 127u) / 128u * 128u; return o; };
  // stream 1's Q descriptors start 1 KB before its images: stream 0's records precede them, so that is valid memory
  for (int s = 0; s < 2; ++s)
    for (int t = 0; t < 3; ++t) m.q[s][t] = p.tier_active[t] ? take(p.qrec_bytes[t]) : 0;
  uint32_t kstage = 0, vstage = 0;
  for (int t = 0; t < 3; ++t) {
    m.kbytes[t] = p.qrec_bytes[t];                     // the K part of a record is laid out like a Q record
    m.vbytes[t] = p.kvrec_bytes[t] - p.qrec_bytes[t];
    if (p.tier_active[t]) { kstage = max(kstage, m.kbytes[t]); vstage = max(vstage, m.vbytes[t]); }
  }
  kstage = (kstage + 127u) / 128u * 128u;
  vstage = (vstage + 127u) / 128u * 128u;
  const uint32_t q_end = cur;
  const uint32_t pbytes = p.tier_active[2] ? 8192u : (p.tier_active[1] ? 4096u : 2048u);
  // ring depths: as deep as shared memory allows (the K ring also serves as the 16 KB output staging tile)
  auto r128 = [](uint32_t b) { return (b + 127u) / 128u * 128u; };
  const uint32_t fixed = 2 * kSets * (pbytes + 512) + 3 * r128(2 * kSets * 64 * 4) + r128(2 * kSets * 2 * 4) +
                         r128(2 * kSets * 64 * 8) + r128(2 * kInfoRing * 16) + r128(2 * B_COUNT * 8);
  const uint32_t budget = q_end + fixed < 232448u ? 232448u - q_end - fixed : 0u;
  // a K block is consumed as soon as a score buffer is free (two per stream), a V block only after the weights of
  // its step are written: the V ring is the deep one
  const int cand[7][2] = {{3, 6}, {3, 5}, {3, 4}, {2, 4}, {2, 3}, {2, 2}, {2, 2}};
  m.nk = 2; m.nv = 2; m.fits = false;
  for (int c = 0; c < 7; ++c) {
    if (2u * (cand[c][0] * kstage + cand[c][1] * vstage) <= budget) {
      m.nk = cand[c][0]; m.nv = cand[c][1]; m.fits = true;
      break;
    }
  }
  while ((uint32_t)m.nk * kstage < 16384u) kstage += 128u;
  m.kstage = kstage; m.vstage = vstage;
  for (int s = 0; s < 2; ++s) {
    for (int g = 0; g < kMaxK; ++g) m.kst[s][g] = g < m.nk ? take(kstage) : 0;
  }
  for (int s = 0; s < 2; ++s)
    for (int g = 0; g < kMaxV; ++g) m.vst[s][g] = g < m.nv ? take(vstage) : 0;
  m.pbytes = pbytes;
  for (int s = 0; s < 2; ++s) for (int g = 0; g < kSets; ++g) m.p[s][g] = take(pbytes);
  for (int s = 0; s < 2; ++s) for (int g = 0; g < kSets; ++g) m.sfp[s][g] = take(512);
  m.factor = take(2 * kSets * 64 * 4);
  m.chg = take(2 * kSets * 2 * 4);
  m.hx = take(2 * kSets * 64 * 8);
  m.href = take(2 * kSets * 64 * 4);
  m.ell = take(2 * kSets * 64 * 4);
  m.info = take(2 * kInfoRing * 16);
  m.bars = take(2 * B_COUNT * 8);
  m.total = cur;
  if (cur > 232448u) m.fits = false;
  return m;
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float lg2(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// packed pairs of fp32 (two lanes per instruction on this architecture) and a three-input maximum
__device__ __forceinline__ uint64_t f2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unf2(uint64_t x, float &lo, float &hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(x)); }
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
// maximum of 16 values in 8 instructions
__device__ __forceinline__ float max16(const float *x) {
  const float m0 = max3(x[0], x[1], x[2]), m1 = max3(x[3], x[4], x[5]), m2 = max3(x[6], x[7], x[8]);
  const float m3 = max3(x[9], x[10], x[11]), m4 = max3(x[12], x[13], x[14]);
  return fmaxf(max3(m0, m1, m2), max3(m3, m4, x[15]));
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
// four floats -> four E2M1 codes in the low 16 bits (x0 in bits 3:0)
__device__ __forceinline__ uint32_t pack_e2m1x4(float x0, float x1, float x2, float x3) {
  uint32_t r;
  asm("{ .reg .b8 a, b; cvt.rn.satfinite.e2m1x2.f32 a, %2, %1; cvt.rn.satfinite.e2m1x2.f32 b, %4, %3; "
      "mov.b32 %0, {a, b, 0, 0}; }"
      : "=r"(r)
      : "f"(x0), "f"(x1), "f"(x2), "f"(x3));
  return r;
}
__device__ __forceinline__ float decode_e4m3(uint32_t c) {
  const __half_raw h = __nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)c, __NV_E4M3);
  return __half2float(*reinterpret_cast<const __half *>(&h));
}

// bounded wait that also gives up as soon as another thread of the CTA has flagged a failure
// (the flag then holds 1 + the shared-memory offset of the barrier that was never completed, for diagnosis)
//
// Waiting warps share their scheduler with the warps doing the softmax arithmetic.  A plain mbarrier.try_wait blocks
// in hardware for a while before it reports failure, so the retry loop issues few instructions (the variant with an
// explicit time hint is expanded into a polling loop with nanosleep and clock reads: more instructions, same run
// time).  The bound is on elapsed clock cycles, checked once per 16 tries.
constexpr long long kWaitLimitCycles = 400000000ll;  // about 0.2 s
__device__ __forceinline__ bool wait_slow(uint64_t *bar, uint32_t parity, volatile int *abort_flag,
                                          long long limit = kWaitLimitCycles) {
  const long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int k = 0; k < 16; ++k)
      if (tc::mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > limit) break;
  }
  atomicCAS(const_cast<int *>(abort_flag), 0, 1 + (int)(tc::smem_u32(bar) & 0xffff));
  return false;
}
__device__ __forceinline__ bool wait_or_abort(uint64_t *bar, uint32_t parity, volatile int *abort_flag,
                                              long long limit = kWaitLimitCycles) {
  if (tc::mbar_try_wait(bar, parity)) return true;
  return wait_slow(bar, parity, abort_flag, limit);
}

// One arrival per warp: every lane's earlier writes are ordered before the elected lane's arrive by the warp barrier.
// (A per-thread arrive is a shared-memory atomic per thread; hundreds of them per step dominate the step time.)
__device__ __forceinline__ void warp_arrive(uint64_t *bar) {
  __syncwarp();
  if ((threadIdx.x & 31) == 0) tc::mbar_arrive(bar);
}

// register rebalancing between warpgroups: the softmax warps hold a whole score row, the others a few scalars
template <int N> __device__ __forceinline__ void reg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void reg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }

__device__ __forceinline__ uint2 ld_shared_volatile_v2(uint32_t saddr) {
  uint2 r;
  asm volatile("ld.volatile.shared.v2.u32 {%0, %1}, [%2];" : "=r"(r.x), "=r"(r.y) : "r"(saddr) : "memory");
  return r;
}

// Valid-slot mask and token index of a block, from the frame's region table (prefix blocks are runs of 64 tokens)
__device__ __forceinline__ unsigned long long table_mask(const Params &p, int a) {
  if (a >= p.R) {
    const int rem = p.P - (a - p.R) * kSlots;
    return rem >= kSlots ? ~0ull : ((1ull << rem) - 1ull);
  }
  return p.region_mask[a % p.R_f];
}
__device__ __forceinline__ long long table_token(const Params &p, int a, int j) {
  if (a >= p.R) return (long long)(a - p.R) * kSlots + j;
  const int t = a / p.R_f, r = a - t * p.R_f;
  return p.P + (long long)t * (p.Hg * p.Wg) + p.region_cell[r * kSlots + j];
}

struct StreamInfo {
  int a;         // query block, or -1
  int n4, n48;   // end of the NVFP4 segment, end of the INT8 segment (list positions)
  int L;
  const uint16_t *ids;
  __device__ __forceinline__ int tier(int i) const { return i < n4 ? 0 : (i < n48 ? 1 : 2); }
};

__device__ __forceinline__ StreamInfo load_stream(const Params &p, int bh, int a) {
  StreamInfo st;
  st.a = a < p.Rt ? a : -1;
  st.n4 = st.n48 = st.L = 0;
  st.ids = nullptr;
  if (a < p.Rt) {
    const int4 c = *reinterpret_cast<const int4 *>(p.counts + ((size_t)bh * p.Rt + a) * 4);
    st.n4 = c.x; st.n48 = c.x + c.y; st.L = c.x + c.y + c.z;
    st.ids = p.ids + (size_t)bh * p.ids_per_head + c.w;
  }
  return st;
}

// ORDERED: the CTA's two query blocks come from the scheduling order of the head (rows of unequal length, HEAD scope);
// otherwise they are blocks 2p and 2p+1 (per-row budgets: every row has the same length, the order is the identity).
// FP4: the plan has an NVFP4 tier.  Without one the exponentiate phase keeps the per-pair interleaved form, which is
// the faster one for the 8-bit and bf16 bodies alone (the compiler's schedule of the unrolled softmax body decides).
template <int D, bool ORDERED, bool FP4, int SETS>
__global__ void __launch_bounds__(Roles<SETS>::NT, 1) attention_kernel(Params p, SmemMap sm, __nv_bfloat16 *__restrict__ out) {
  constexpr int kSets = SETS, NT = Roles<SETS>::NT, kSoftmaxWarps = Roles<SETS>::kSoftmaxWarps;
  constexpr int kMmaWarp0 = Roles<SETS>::kMmaWarp0, kPvWarp0 = Roles<SETS>::kPvWarp0, kLoadWarp0 = Roles<SETS>::kLoadWarp0;
  constexpr int kShift = Roles<SETS>::kShift, kMask = Roles<SETS>::kMask;
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_abort;

  const int tid = threadIdx.x, lane = tid & 31;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);  // warp-uniform by construction
  const int R = p.R, Rt = p.Rt, pairs = (Rt + 1) / 2;
  const int bh = blockIdx.x / pairs, pr = blockIdx.x % pairs;
  __nv_bfloat16 *out_head = out + (size_t)bh * p.Ntot * D;
  // the two query blocks of this CTA: equally long rows of the head (scheduling order written with the lists)
  int a0 = 2 * pr, a1 = 2 * pr + 1;
  if (ORDERED) {
    const uint16_t *ord = p.order + ((size_t)bh * pairs + pr) * 2;
    a0 = ord[0];
    a1 = ord[1];
  }
  const StreamInfo st0 = load_stream(p, bh, a0), st1 = load_stream(p, bh, a1);

  uint64_t *bars = reinterpret_cast<uint64_t *>(smem + sm.bars);
  auto bar = [&](int s, int which) -> uint64_t * { return bars + s * B_COUNT + which; };
  float *s_factor = reinterpret_cast<float *>(smem + sm.factor);      // [s][set][64]
  uint32_t *s_chg = reinterpret_cast<uint32_t *>(smem + sm.chg);      // [s][set][2]
  uint2 *s_hx = reinterpret_cast<uint2 *>(smem + sm.hx);              // [s][set][64]
  float *s_href = reinterpret_cast<float *>(smem + sm.href);          // [s][set][64]
  float *s_ell = reinterpret_cast<float *>(smem + sm.ell);            // [s][set][64]
  uint8_t *s_info = smem + sm.info;                                   // [s][kInfoRing] 16 bytes

  for (int k_ = tid; k_ < 2 * kSets * 64; k_ += NT) s_hx[k_] = make_uint2(0u, 0xffffffffu);  // no step has this tag
  if (warp == 0) {
    tc::tmem_alloc(&s_tmem_base, kTmemCols);
    tc::tmem_relinquish();
  }
  if (tid == 32) {
    for (int s = 0; s < 2; ++s) {
      for (int g = 0; g < 2; ++g) tc::mbar_init(bar(s, B_SFREE + g), 2);
      for (int g = 0; g < kSets; ++g) {
        tc::mbar_init(bar(s, B_SREADY + g), 1);
        tc::mbar_init(bar(s, B_PREADY + g), 2);  // the two softmax warps of the step (P written)
        tc::mbar_init(bar(s, B_PVDONE + g), 1);
        tc::mbar_init(bar(s, B_CORROK + g), 4);  // the stream's four correction warps (accumulator rescaled)
      }
      for (int g = 0; g < kMaxK; ++g) {
        tc::mbar_init(bar(s, B_FULLK + g), 1);
        tc::mbar_init(bar(s, B_KFREE + g), 1);
      }
      for (int g = 0; g < kMaxV; ++g) {
        tc::mbar_init(bar(s, B_FULLV + g), 1);
        tc::mbar_init(bar(s, B_VFREE + g), 1);
      }
      tc::mbar_init(bar(s, B_ELL), 2 * kSets);
      tc::mbar_init(bar(s, B_Q), 1);
    }
    tc::fence_barrier_init();
    s_abort = 0;
  }
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tmem = s_tmem_base;
  volatile int *abortp = &s_abort;

  // =========================================================================================== softmax warps
  if (warp < kSoftmaxWarps) {
    reg_inc<(SETS == 4 ? 88 : 128)>();
    // The warps w, w+4, w+8, ... share a scheduler and own the same 32 query rows; they take the steps of their sets
    // in turn, one thread per full 64-key row: while one exponentiates and packs its step (special-function bound),
    // the others fetch, mask and reduce later ones.  The only hand-off between them is the running maximum.
    const int s = (warp & 3) >> 1, set = warp >> 2;
    const int r = (warp & 1) * 32 + lane;  // query row inside the stream's block
    const StreamInfo S = s ? st1 : st0;
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    const float gqk = p.gscale[bh * 4 + 0] * p.gscale[bh * 4 + 1] * p.scale * kLog2e;
    const float dq8s = (S.a >= 0 && S.a < R && p.tier_active[1]) ? p.dq8[(size_t)bh * R + S.a] * p.scale * kLog2e : 0.f;
    const float c16 = p.scale * kLog2e;
    float h_own = -INFINITY, ell = 0.f;  // log2-domain maximum after this warp's last step; its partial denominator
    const int g = set;                   // P buffer, barriers and hand-off slot of this set
    uint2 *my_hx = s_hx + (s * kSets + set) * 64 + r;                // running maximum after my steps, tagged with the step
    const uint32_t prev_hx = tc::smem_u32(s_hx + (s * kSets + ((set + kSets - 1) % kSets)) * 64 + r);
    uint8_t *prow = smem + sm.p[s][g] + r * 16;

    for (int i = set; i < S.L; i += kSets) {
      const int tier = S.tier(i);
      const uint32_t kp = (uint32_t)(i >> kShift) & 1u;  // completion parity of this set's k-th step
      const uint32_t s_col = tmem + lane_addr + col_s(s, i & 1);
      if (!wait_or_abort(bar(s, B_SREADY + g), kp, abortp)) break;
      tc::fence_after_sync();
      // the step's mask and key scale (written before its K block was requested) are read while the scores load
      const uint8_t *info = s_info + (s * kInfoRing + (i & (kInfoRing - 1))) * 16;
      const uint2 kmask = *reinterpret_cast<const uint2 *>(info);
      float coef;
      if (tier == 2) coef = c16;
      else if (tier == 1) coef = dq8s * *reinterpret_cast<const float *>(info + 8);
      else coef = gqk;
      float v[64];
      {
        uint32_t a0[16], a1[16], a2[16], a3[16];
        tc::tmem_ld16(s_col, a0);
        tc::tmem_ld16(s_col + 16, a1);
        tc::tmem_ld16(s_col + 32, a2);
        tc::tmem_ld16(s_col + 48, a3);
        tc::wait_ld();
        // int32 accumulators become floats exactly through a magic-number add and subtract (|S| < 2^22): two
        // full-rate operations instead of a conversion on the special-function unit
        if (tier == 1) {
          const uint64_t moff = f2(-12582912.0f, -12582912.0f);
#pragma unroll
          for (int c = 0; c < 16; c += 2) {
            unf2(add2(f2(__uint_as_float(a0[c] + 0x4B400000u), __uint_as_float(a0[c + 1] + 0x4B400000u)), moff), v[c], v[c + 1]);
            unf2(add2(f2(__uint_as_float(a1[c] + 0x4B400000u), __uint_as_float(a1[c + 1] + 0x4B400000u)), moff), v[16 + c], v[17 + c]);
            unf2(add2(f2(__uint_as_float(a2[c] + 0x4B400000u), __uint_as_float(a2[c + 1] + 0x4B400000u)), moff), v[32 + c], v[33 + c]);
            unf2(add2(f2(__uint_as_float(a3[c] + 0x4B400000u), __uint_as_float(a3[c + 1] + 0x4B400000u)), moff), v[48 + c], v[49 + c]);
          }
        } else {
#pragma unroll
          for (int c = 0; c < 16; ++c) {
            v[c] = __uint_as_float(a0[c]); v[16 + c] = __uint_as_float(a1[c]);
            v[32 + c] = __uint_as_float(a2[c]); v[48 + c] = __uint_as_float(a3[c]);
          }
        }
      }
      tc::fence_before_sync();
      warp_arrive(bar(s, B_SFREE + (i & 1)));
      if ((kmask.x & kmask.y) != 0xffffffffu) {  // padding keys take no part
        if (kmask.x == 0xffffffffu && kmask.y == 0x7fffffffu) {
          v[63] = -INFINITY;  // a region of 63 tokens (the balanced partition's common case): one padding slot
        } else if (kmask.x == 0xffffffffu) {
#pragma unroll
          for (int c = 0; c < 32; ++c) v[32 + c] = ((kmask.y >> c) & 1u) ? v[32 + c] : -INFINITY;
        } else {  // ragged edge tile
#pragma unroll
          for (int c = 0; c < 32; ++c) {
            v[c] = ((kmask.x >> c) & 1u) ? v[c] : -INFINITY;
            v[32 + c] = ((kmask.y >> c) & 1u) ? v[32 + c] : -INFINITY;
          }
        }
      }
      // maxima of the four 16-key groups (pairwise trees), then of the row
      float gm[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) gm[q] = max16(v + q * 16);
      const float pmax = fmaxf(max3(gm[0], gm[1], gm[2]), gm[3]) * coef;  // log2 domain
      // PV(i-4) done: this set's P buffer is free and the correction warps are past step i-4
      if (i >= kSets && !wait_or_abort(bar(s, B_PVDONE + g), (kp ^ 1u), abortp)) break;
      // running maximum after step i-1: the thread that owns this row in the previous set leaves it, tagged with its
      // step, in shared memory (one 8-byte store, one 8-byte load: no barrier on this chain)
      float h_prev = -INFINITY;
      if (i > 0) {
        uint2 hv = ld_shared_volatile_v2(prev_hx);
        for (uint32_t spin = 0; hv.y != (uint32_t)(i - 1); ++spin) {
          if ((spin & 1023u) == 1023u && (*abortp || spin > (1u << 24))) break;
          hv = ld_shared_volatile_v2(prev_hx);
        }
        const bool got = hv.y == (uint32_t)(i - 1);
        if (!__all_sync(0xffffffffu, got)) {
          atomicCAS(const_cast<int *>(abortp), 0, 1 + (int)(tc::smem_u32(bar(s, B_CORROK)) & 0xffff));
          break;
        }
        h_prev = __uint_as_float(hv.x);
      }
      const float m_new = fmaxf(h_prev, pmax);
      *my_hx = make_uint2(__float_as_uint(m_new), (uint32_t)i);
      s_factor[(s * kSets + g) * 64 + r] = ex2(h_prev - m_new);  // 0 on the first block (h_prev = -inf)
      const uint32_t moved = __ballot_sync(0xffffffffu, m_new != h_prev);
      if (lane == 0) s_chg[(s * kSets + g) * 2 + (warp & 1)] = moved;
      ell *= ex2(h_own - m_new);
      h_own = m_new;

      const uint64_t coef2 = f2(coef, coef);
      if (!FP4 && tier == 2) {
        const uint64_t bias2 = f2(-m_new, -m_new);
        uint64_t sum2 = 0;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          uint32_t w4[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            float t0, t1;
            unf2(fma2(f2(v[c * 8 + 2 * j], v[c * 8 + 2 * j + 1]), coef2, bias2), t0, t1);
            const float w0 = ex2(t0), w1 = ex2(t1);
            sum2 = add2(sum2, f2(w0, w1));
            w4[j] = pack_bf16x2(w0, w1);
          }
          *reinterpret_cast<uint4 *>(prow + c * 1024) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
        }
        float s0, s1;
        unf2(sum2, s0, s1);
        ell += s0 + s1;
      } else if (!FP4) {
        const uint64_t bias2 = f2(kOffsetP8 - m_new, kOffsetP8 - m_new);
        uint64_t sum2 = 0;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t w4[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            float t0, t1, t2, t3;
            unf2(fma2(f2(v[c * 16 + 4 * j + 0], v[c * 16 + 4 * j + 1]), coef2, bias2), t0, t1);
            unf2(fma2(f2(v[c * 16 + 4 * j + 2], v[c * 16 + 4 * j + 3]), coef2, bias2), t2, t3);
            const float w0 = ex2(t0), w1 = ex2(t1), w2 = ex2(t2), w3 = ex2(t3);
            sum2 = add2(add2(sum2, f2(w0, w1)), f2(w2, w3));
            w4[j] = pack_e4m3x2(w0, w1) | (pack_e4m3x2(w2, w3) << 16);
          }
          *reinterpret_cast<uint4 *>(prow + c * 1024) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
        }
        float s0, s1;
        unf2(sum2, s0, s1);
        ell += kEtaP8 * (s0 + s1);  // the denominator sums the amplified fp32 weights; eta restores the unit
      } else if (tier != 0) {
        // the scores of the row become the exponent arguments, then the weights, in place: all 64 exponentials are
        // issued before any is consumed (the 8-bit path carries the 2^8.807 offset in the exponent)
        const float b = tier == 1 ? kOffsetP8 - m_new : -m_new;
        const uint64_t bias2 = f2(b, b);
#pragma unroll
        for (int j = 0; j < 32; ++j) unf2(fma2(f2(v[2 * j], v[2 * j + 1]), coef2, bias2), v[2 * j], v[2 * j + 1]);
#pragma unroll
        for (int j = 0; j < 64; ++j) v[j] = ex2(v[j]);
        uint64_t sum2 = 0;
#pragma unroll
        for (int j = 0; j < 32; j += 2) sum2 = add2(sum2, add2(f2(v[2 * j], v[2 * j + 1]), f2(v[2 * j + 2], v[2 * j + 3])));
        float s0, s1;
        unf2(sum2, s0, s1);
        if (tier == 2) {
#pragma unroll
          for (int c = 0; c < 8; ++c)
            *reinterpret_cast<uint4 *>(prow + c * 1024) =
                make_uint4(pack_bf16x2(v[c * 8 + 0], v[c * 8 + 1]), pack_bf16x2(v[c * 8 + 2], v[c * 8 + 3]),
                           pack_bf16x2(v[c * 8 + 4], v[c * 8 + 5]), pack_bf16x2(v[c * 8 + 6], v[c * 8 + 7]));
          ell += s0 + s1;
        } else {
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            uint32_t w4[4];
#pragma unroll
            for (int j = 0; j < 4; ++j)
              w4[j] = pack_e4m3x2(v[c * 16 + 4 * j], v[c * 16 + 4 * j + 1]) |
                      (pack_e4m3x2(v[c * 16 + 4 * j + 2], v[c * 16 + 4 * j + 3]) << 16);
            *reinterpret_cast<uint4 *>(prow + c * 1024) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
          }
          ell += kEtaP8 * (s0 + s1);  // the denominator sums the amplified fp32 weights; eta restores the unit
        }
      } else {
        // Group scales from each group's largest weight (Eq. "v2-nvfp4-probability"), folded into the exponent:
        // sigma = E4M3(448 * max w); scaled weight u = w * 2688 / sigma = 2^(x - m + log2(2688) - log2(sigma)).
        // The four scale chains run first (interleaved), then the exponentials in batches of 32 that are all issued
        // before any is consumed.
        uint32_t sfword = 0;
        float bb[4], sl[4];
        bool live[4];
#pragma unroll
        for (int gi = 0; gi < 4; ++gi) {
          const float gw = ex2(fmaf(gm[gi], coef, -m_new));
          const uint32_t sc = pack_e4m3x2(__fmul_rn(448.0f, gw), 0.f) & 0xffu;
          sfword |= sc << (8 * gi);
          // E4M3 code -> fp32: for normal codes the bit pattern is a shift and a re-bias; the 7 subnormal codes
          // and zero (weights below 2^-15 of the row maximum) take the general conversion
          const float sigma = sc >= 8u ? __uint_as_float((sc << 20) + 0x3C000000u) : decode_e4m3(sc);
          live[gi] = sc != 0u;
          bb[gi] = (live[gi] ? 11.392317422778762f - lg2(sigma) : 0.f) - m_new;  // log2(2688) = 11.3923...
          sl[gi] = live[gi] ? sigma * (1.0f / 2688.0f) : 1.0f;
        }
        *reinterpret_cast<uint32_t *>(smem + sm.sfp[s][g] + (r & 31) * 16 + (r >> 5) * 4) = sfword;
        {
          // the scores of the row become the exponent arguments, then the scaled weights, in place
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const float b = bb[j >> 3];
            unf2(fma2(f2(v[2 * j], v[2 * j + 1]), coef2, f2(b, b)), v[2 * j], v[2 * j + 1]);
          }
#pragma unroll
          for (int j = 0; j < 64; ++j) v[j] = ex2(v[j]);
#pragma unroll
          for (int gp = 0; gp < 2; ++gp) {  // 32 keys = two groups = one 16-byte chunk of the row
            uint32_t cw[4];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              const float *x = v + gp * 32 + h * 16;
              const uint64_t sa = add2(f2(x[0], x[1]), f2(x[2], x[3])), sb = add2(f2(x[4], x[5]), f2(x[6], x[7]));
              const uint64_t sc2 = add2(f2(x[8], x[9]), f2(x[10], x[11])), sd = add2(f2(x[12], x[13]), f2(x[14], x[15]));
              float s0, s1;
              unf2(add2(add2(sa, sb), add2(sc2, sd)), s0, s1);
              ell = fmaf(s0 + s1, sl[gp * 2 + h], ell);
              const uint32_t c0 = pack_e2m1x4(x[0], x[1], x[2], x[3]) | (pack_e2m1x4(x[4], x[5], x[6], x[7]) << 16);
              const uint32_t c1 = pack_e2m1x4(x[8], x[9], x[10], x[11]) | (pack_e2m1x4(x[12], x[13], x[14], x[15]) << 16);
              cw[h * 2 + 0] = live[gp * 2 + h] ? c0 : 0u;
              cw[h * 2 + 1] = live[gp * 2 + h] ? c1 : 0u;
            }
            *reinterpret_cast<uint4 *>(prow + gp * 1024) = make_uint4(cw[0], cw[1], cw[2], cw[3]);
          }
        }
      }
      tc::fence_async_smem();
      warp_arrive(bar(s, B_PREADY + g));
    }
    if (S.L > 0) {
      s_ell[(s * kSets + set) * 64 + r] = ell;
      s_href[(s * kSets + set) * 64 + r] = h_own;  // reference of this partial denominator
      warp_arrive(bar(s, B_ELL));
    }
  }
  // =========================================================================================== loader warps
  else {
  reg_dec<40>();
  if (warp >= kLoadWarp0) {
    // Warps kLoadWarp0 + s request the K blocks of stream s (and its Q records), warps kLoadWarp0 + 2 + s its V
    // blocks: a K block is consumed as soon as a score buffer is free, a V block only once the weights of its step
    // are written, several steps later, so the two rings advance independently.
    // Warp-uniform loop.  Lane l holds list entry 32 * batch + l ready for use: the record's address, the valid-key
    // mask and the INT8 key scale; the ids of the next two batches and the scales of the next one are already on
    // their way while a batch is used, so that a step costs a few shuffles and the copy request of one elected lane.
    const int s = (warp - kLoadWarp0) & 1;
    const bool is_v = warp >= kLoadWarp0 + 2;
    StreamInfo S = s ? st1 : st0;
    S.n4 = __shfl_sync(0xffffffffu, S.n4, 0);
    S.n48 = __shfl_sync(0xffffffffu, S.n48, 0);
    S.L = __shfl_sync(0xffffffffu, S.L, 0);
    if (S.L > 0) {
      if (!is_v && tc::elect_one()) {
        const int nn[3] = {S.n4, S.n48 - S.n4, S.L - S.n48};
        uint32_t bytes = 0;
        for (int t = 0; t < 3; ++t) if (nn[t] > 0) bytes += p.qrec_bytes[t];
        tc::mbar_arrive_expect_tx(bar(s, B_Q), bytes);
        for (int t = 0; t < 3; ++t)
          if (nn[t] > 0)
            tc::bulk_g2s(smem + sm.q[s][t], p.qrec[t] + ((size_t)bh * rec_blocks(p, t) + S.a) * p.qrec_bytes[t], p.qrec_bytes[t],
                         bar(s, B_Q));
      }
      __syncwarp();
      const size_t head_blocks = (size_t)bh * R;
      auto list_id = [&](int idx) -> int {
        int b = idx < S.L ? (int)S.ids[idx] : 0;
        if (b >= Rt) { atomicExch(p.status, kDevBadList); b = 0; }
        return b;
      };
      auto key_scale = [&](int idx, int b) -> float {
        return (!is_v && idx < S.L && S.tier(idx) == 1) ? p.dk8[head_blocks + b] : 0.f;
      };
      auto record = [&](int idx, int b) -> unsigned long long {
        const int t = S.tier(idx);
        return reinterpret_cast<unsigned long long>(p.kvrec[t] + ((size_t)bh * rec_blocks(p, t) + b) * p.kvrec_bytes[t] +
                                                    (is_v ? sm.kbytes[t] : 0u));
      };
      // batch -1 is empty: the loop's refill at "src == 31" then also serves the first batch
      int nxt_b = list_id(lane), nn_b = list_id(32 + lane);
      float cur_dk = 0.f, nxt_dk = key_scale(lane, nxt_b);
      unsigned long long cur_rec = 0, cur_mask = 0;
      const uint32_t nb0 = is_v ? sm.vbytes[0] : sm.kbytes[0], nb1 = is_v ? sm.vbytes[1] : sm.kbytes[1],
                     nb2 = is_v ? sm.vbytes[2] : sm.kbytes[2];
      uint8_t *dst = smem + (is_v ? sm.vst[s][0] : sm.kst[s][0]);
      const uint32_t stage = is_v ? sm.vstage : sm.kstage;
      const int depth = is_v ? sm.nv : sm.nk;
      const int b_full = is_v ? B_FULLV : B_FULLK, b_free = is_v ? B_VFREE : B_KFREE;
      int kk = 0;         // ring slot
      uint32_t kpar = 1;  // parity of the consumption that frees the slot (first pass: nothing to wait for)
      bool kwrapped = false;
      for (int i = -1; i < S.L; ++i) {
        const int src = i & 31;
        if (i >= 0) {
        const uint32_t rlo = __shfl_sync(0xffffffffu, (uint32_t)cur_rec, src);
        const uint32_t rhi = __shfl_sync(0xffffffffu, (uint32_t)(cur_rec >> 32), src);
        const uint32_t mlo = __shfl_sync(0xffffffffu, (uint32_t)cur_mask, src);
        const uint32_t mhi = __shfl_sync(0xffffffffu, (uint32_t)(cur_mask >> 32), src);
        const float dk = __shfl_sync(0xffffffffu, cur_dk, src);
        const uint8_t *rec = reinterpret_cast<const uint8_t *>(((unsigned long long)rhi << 32) | rlo);
        const uint32_t nb = i < S.n4 ? nb0 : (i < S.n48 ? nb1 : nb2);
        if (kwrapped && !wait_or_abort(bar(s, b_free + kk), kpar, abortp)) break;
        if (tc::elect_one()) {
          // the step's mask and key scale enter the info ring before the data the softmax waits for is requested
          if (!is_v)
            *reinterpret_cast<uint4 *>(s_info + (s * kInfoRing + (i & (kInfoRing - 1))) * 16) =
                make_uint4(mlo, mhi, __float_as_uint(dk), 0u);
          tc::mbar_arrive_expect_tx(bar(s, b_full + kk), nb);
          tc::bulk_g2s(dst + kk * stage, rec, nb, bar(s, b_full + kk));
        }
        __syncwarp();
        if (++kk == depth) { kk = 0; kpar ^= 1u; kwrapped = true; }
        }
        if (src == 31) {  // next batch: its ids and scales were requested one batch ago
          const int b = nxt_b;
          cur_dk = nxt_dk;
          cur_rec = record(i + 1 + lane, b);
          cur_mask = table_mask(p, b);
          nxt_b = nn_b;
          nxt_dk = key_scale(i + 33 + lane, nxt_b);
          nn_b = list_id(i + 65 + lane);
        }
      }
    }
  }
  // =========================================================================================== MMA warps
  else if (warp >= kMmaWarp0 && warp < kPvWarp0) {
    // The whole warp runs this loop with warp-uniform control flow and values; only the tcgen05 instructions
    // themselves are issued by one elected lane.  (Under a lane-0 branch every descriptor would have to be moved from
    // vector to uniform registers before each issue, which costs more than the MMA itself.)
    const int s = warp - kMmaWarp0;
    StreamInfo S = s ? st1 : st0;
    S.n4 = __shfl_sync(0xffffffffu, S.n4, 0);
    S.n48 = __shfl_sync(0xffffffffu, S.n48, 0);
    S.L = __shfl_sync(0xffffffffu, S.L, 0);
    if (S.L > 0 && wait_or_abort(bar(s, B_Q), 0, abortp)) {
      // operand descriptors, built once; inside the loop only the 16-byte-unit start address (low bits) moves
      const uint64_t qd0 = tc::smem_desc(tc::smem_u32(smem + sm.q[s][0]) - (s ? 1024u : 0u), 1024, 128);
      const uint64_t qd1 = tc::smem_desc(tc::smem_u32(smem + sm.q[s][1]) - (s ? 1024u : 0u), 1024, 128);
      const uint64_t qd2 = tc::smem_desc(tc::smem_u32(smem + sm.q[s][2]) - (s ? 1024u : 0u), 1024, 128);
      const uint64_t kd0 = tc::smem_desc(tc::smem_u32(smem + sm.kst[s][0]), 1024, 128);
      const uint64_t ksf0 = tc::smem_desc(tc::smem_u32(smem + sm.kst[s][0]) + kSlots * D / 2, 128, 128);
      const uint32_t kstep = sm.kstage >> 4;
      const uint32_t t_sfq = tmem + col_sfq(s), t_sfk = tmem + col_sfk(s);
      if (S.n4 > 0) {  // Q scale factors go to TMEM once; the record carries them for rows 0..63 and again for rows
                       // 64..127, so the same atom serves either stream
        if (tc::elect_one()) {
#pragma unroll
          for (int k = 0; k < D / 64; ++k)
            tc::tmem_cp_sf(t_sfq + 4 * k, tc::smem_desc(tc::smem_u32(smem + sm.q[s][0]) + kSlots * D / 2 + k * kSfAtomBytes,
                                                         128, 128));
        }
      }
      int kk = 0;
      uint32_t kpar = 0;
      // the score tiles are double buffered, so Q K^T runs up to two steps ahead of the softmax
      for (int j = 0; j < S.L; ++j) {
        const int g = j & 1;
        if (!wait_or_abort(bar(s, B_FULLK + kk), kpar, abortp)) break;
        if (!wait_or_abort(bar(s, B_SFREE + g), ((j >> 1) & 1) ^ 1, abortp)) break;
        tc::fence_after_sync();
        const uint64_t kd = kd0 + (uint64_t)(kk * kstep);
        const uint32_t d_s = tmem + col_s(s, g);
        if (tc::elect_one()) {
          if (j >= S.n48) {
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) tc::mma_f16(d_s, qd2 + ks * 128, kd + ks * 128, tc::idesc_bf16(64), ks > 0);
          } else if (j >= S.n4) {
#pragma unroll
            for (int ks = 0; ks < D / 32; ++ks) tc::mma_i8(d_s, qd1 + ks * 128, kd + ks * 128, tc::idesc_i8(64), ks > 0);
          } else {
            const uint64_t ksf = ksf0 + (uint64_t)(kk * kstep);
#pragma unroll
            for (int k = 0; k < D / 64; ++k) tc::tmem_cp_sf(t_sfk + 4 * k, ksf + k * (kSfAtomBytes >> 4));
#pragma unroll
            for (int ks = 0; ks < D / 64; ++ks)
              tc::mma_nvfp4(d_s, qd0 + ks * 128, kd + ks * 128, tc::idesc_nvfp4(64), ks > 0, t_sfq + 4 * ks, t_sfk + 4 * ks);
          }
          tc::mma_commit(bar(s, B_SREADY + (j & kMask)));
          tc::mma_commit(bar(s, B_KFREE + kk));
        }
        __syncwarp();
        if (++kk == sm.nk) { kk = 0; kpar ^= 1u; }
      }
    }
  }
  // =========================================================================================== PV warps
  else if (warp >= kPvWarp0) {
    const int s = warp - kPvWarp0;
    StreamInfo S = s ? st1 : st0;
    S.n4 = __shfl_sync(0xffffffffu, S.n4, 0);
    S.n48 = __shfl_sync(0xffffffffu, S.n48, 0);
    S.L = __shfl_sync(0xffffffffu, S.L, 0);
    if (S.L > 0) {
      const uint64_t vd0 = tc::smem_desc(tc::smem_u32(smem + sm.vst[s][0]), D * 16, 128);
      const uint64_t vsf0 = tc::smem_desc(tc::smem_u32(smem + sm.vst[s][0]) + D * kSlots / 2, 128, 128);
      const uint64_t pd0 = tc::smem_desc(tc::smem_u32(smem + sm.p[s][0]), 1024, 128);
      const uint64_t sfpd0 = tc::smem_desc(tc::smem_u32(smem + sm.sfp[s][0]), 128, 128);
      const uint32_t pstep = sm.pbytes >> 4;
      const uint32_t vstep = sm.vstage >> 4;
      const uint32_t t_sfv = tmem + col_sfv(s), t_sfp = tmem + col_sfp(s), t_o = tmem + col_o(s);
      int vv = 0;
      uint32_t vpar = 0;
      for (int j = 0; j < S.L; ++j) {
        // ---- O^T += V(j)^T P(j)^T, once P(j) is written and the accumulator is rescaled for step j
        const int g = j & kMask;
        if (!wait_or_abort(bar(s, B_FULLV + vv), vpar, abortp)) break;
        // P(j) is written and the stream's correction warps have rescaled the accumulator where step j asked for it
        if (!wait_or_abort(bar(s, B_CORROK + g), (j >> kShift) & 1, abortp)) break;
        tc::fence_after_sync();
        const uint64_t vd = vd0 + (uint64_t)(vv * vstep);
        const uint64_t pdg = pd0 + (uint64_t)(g * pstep), sfpdg = sfpd0 + (uint64_t)(g * 32);
        const uint32_t acc = j > 0;
        if (tc::elect_one()) {
          if (j >= S.n48) {
#pragma unroll
            for (int ks = 0; ks < 4; ++ks)
              tc::mma_f16(t_o, vd + ks * (2 * D), pdg + ks * 128, tc::idesc_bf16(64), acc | (ks > 0));
          } else if (j >= S.n4) {
#pragma unroll
            for (int ks = 0; ks < 2; ++ks)
              tc::mma_f8f6f4(t_o, vd + ks * (2 * D), pdg + ks * 128, tc::idesc_e4m3(64), acc | (ks > 0));
          } else {
            tc::tmem_cp_sf(t_sfv, vsf0 + (uint64_t)(vv * vstep));
            tc::tmem_cp_sf(t_sfp, sfpdg);
            tc::mma_nvfp4(t_o, vd, pdg, tc::idesc_nvfp4(64), acc, t_sfv, t_sfp);
          }
          tc::mma_commit(bar(s, B_PVDONE + g));
          tc::mma_commit(bar(s, B_VFREE + vv));
        }
        __syncwarp();
        if (++vv == sm.nv) { vv = 0; vpar ^= 1u; }
      }
    }
  }
  // =========================================================================================== correction warps
  else {
    const int s = (warp - kSoftmaxWarps) >> 2;  // four correction warps per stream
    const int cw = (warp - kSoftmaxWarps) & 3;  // lane quarter
    const int ch = cw * 32 + lane;              // channel (TMEM lane)
    const uint32_t lane_addr = (uint32_t)(cw * 32) << 16;
    const float gv = p.gscale[bh * 4 + 2];
    const float dv8 = (p.tier_active[1] && ch < D) ? p.dv8[(size_t)bh * D + ch] : 0.f;
    auto unit_of = [&](int t) -> float {  // common units per accumulator unit, for this thread's channel
      return t == 0 ? __fdiv_rn(gv, 2688.0f) : (t == 1 ? kEtaP8 * dv8 : 1.0f);
    };
    const StreamInfo &S = s ? st1 : st0;
    // Every step passes through these warps between the softmax and the product: once P(i) is written they read the
    // step's "maximum moved" ballots and, only if one is set or the segment changes, wait for product i-1 and rescale
    // their lane quarter of the accumulator; then they let product i go.  Most steps move no maximum.
    for (int i = 0; i < S.L; ++i) {
      const int g = i & kMask;
      if (!wait_or_abort(bar(s, B_PREADY + g), (i >> kShift) & 1, abortp)) break;
      const bool tier_switch = (i == S.n4) || (i == S.n48);
      const uint2 moved = ld_shared_volatile_v2(tc::smem_u32(s_chg + (s * kSets + g) * 2));
      if (i == 0 || ((moved.x | moved.y) == 0u && !tier_switch)) {
        if (lane == 0) tc::mbar_arrive(bar(s, B_CORROK + g));
        continue;
      }
      const int tier = S.tier(i);
      // everything that does not need the accumulator comes before the wait for product i-1
      float lane_factor = 1.0f;
      if (tier_switch && ch < D) {
        const float un = unit_of(tier), up = unit_of(S.tier(i - 1));
        lane_factor = un > 0.f ? __fdiv_rn(up, un) : 0.f;
      }
      const float *fac = s_factor + (s * kSets + g) * 64;
      // column groups (eight queries each) with a moved maximum; all of them when the segment changes.  Two groups
      // are in flight at a time: their loads are issued together, so a rescale costs one TMEM round trip per pair.
      uint32_t todo = 0;
#pragma unroll
      for (int c = 0; c < 8; ++c)
        if (tier_switch || (((c < 4 ? moved.x : moved.y) >> ((c & 3) * 8)) & 0xffu) != 0u) todo |= 1u << c;
      if (!wait_or_abort(bar(s, B_PVDONE + ((i - 1) & kMask)), ((i - 1) >> kShift) & 1, abortp)) break;
      tc::fence_after_sync();
#pragma unroll 1
      while (todo) {
        const int c0 = __ffs(todo) - 1;
        todo &= todo - 1;
        const int c1 = todo ? __ffs(todo) - 1 : -1;
        if (c1 >= 0) todo &= todo - 1;
        uint32_t o0[8], o1[8];
        tc::tmem_ld8(tmem + lane_addr + col_o(s) + c0 * 8, o0);
        if (c1 >= 0) tc::tmem_ld8(tmem + lane_addr + col_o(s) + c1 * 8, o1);
        tc::wait_ld();
#pragma unroll
        for (int j = 0; j < 8; ++j) o0[j] = __float_as_uint(__uint_as_float(o0[j]) * (fac[c0 * 8 + j] * lane_factor));
        tc::tmem_st8(tmem + lane_addr + col_o(s) + c0 * 8, o0);
        if (c1 >= 0) {
#pragma unroll
          for (int j = 0; j < 8; ++j) o1[j] = __float_as_uint(__uint_as_float(o1[j]) * (fac[c1 * 8 + j] * lane_factor));
          tc::tmem_st8(tmem + lane_addr + col_o(s) + c1 * 8, o1);
        }
      }
      tc::wait_st();
      tc::fence_before_sync();
      warp_arrive(bar(s, B_CORROK + g));
    }
    // ---------------------------------------------------------- epilogue: O = U / l, back to raster order
    if (S.a >= 0) {
      const unsigned long long qmask = table_mask(p, S.a);
      uint16_t *stage = reinterpret_cast<uint16_t *>(smem + sm.kst[s][0]);  // [64][D] bf16 over the K ring
      bool ok = S.L > 0 && !*abortp;
      if (ok) ok = wait_or_abort(bar(s, B_ELL), 0, abortp);
      if (ok) ok = wait_or_abort(bar(s, B_PVDONE + ((S.L - 1) & kMask)), ((S.L - 1) >> kShift) & 1, abortp);
      const int ltid = tid - (kSoftmaxWarps + 4 * s) * 32;  // thread index inside the stream's correction group
      float *s_inv = s_factor + (s * kSets) * 64;            // 1 / l per query (the factors are no longer needed)
      if (ok && ltid < 64) {
        // the sets of a row kept partial denominators relative to their own last maximum
        float hf = -INFINITY, l = 0.f;
#pragma unroll 1
        for (int k = 0; k < kSets; ++k) hf = fmaxf(hf, s_href[(s * kSets + k) * 64 + ltid]);
#pragma unroll 1
        for (int k = 0; k < kSets; ++k) {  // a set without a step has ell = 0 and reference -inf
          const float lk = s_ell[(s * kSets + k) * 64 + ltid];
          if (lk > 0.f) l += lk * ex2(s_href[(s * kSets + k) * 64 + ltid] - hf);
        }
        s_inv[ltid] = l > 0.f ? __fdiv_rn(1.0f, l) : 0.f;
      }
      if (s == 0) asm volatile("bar.sync 1, 128;" ::: "memory"); else asm volatile("bar.sync 2, 128;" ::: "memory");
      if (ok) {
        tc::fence_after_sync();
        const float unit = ch < D ? unit_of(S.tier(S.L - 1)) : 0.f;
#pragma unroll 1
        for (int c = 0; c < 8; ++c) {
          uint32_t o[8];
          tc::tmem_ld8(tmem + lane_addr + col_o(s) + c * 8, o);
          tc::wait_ld();
          if (ch < D) {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const int qr = c * 8 + j;
              const float inv = s_inv[qr];
              const float val = inv > 0.f ? __uint_as_float(o[j]) * unit * inv : 0.f;
              stage[qr * D + ch] = __bfloat16_as_ushort(__float2bfloat16_rn(val));
            }
          }
        }
      } else if (S.L == 0) {  // rows without a retained key return zero (App. C.1)
        for (int idx = ltid; idx < kSlots * (D / 8); idx += 128) reinterpret_cast<uint4 *>(stage)[idx] = make_uint4(0, 0, 0, 0);
      }
      if (s == 0) asm volatile("bar.sync 1, 128;" ::: "memory"); else asm volatile("bar.sync 2, 128;" ::: "memory");
      if (ok || S.L == 0) {
#pragma unroll 1
        for (int idx = ltid; idx < kSlots * (D / 8); idx += 128) {
          const int j = idx / (D / 8), c8 = idx % (D / 8);
          if ((qmask >> j) & 1ull)
            *reinterpret_cast<uint4 *>(out_head + (size_t)table_token(p, S.a, j) * D + c8 * 8) =
                *reinterpret_cast<const uint4 *>(stage + j * D + c8 * 8);
        }
      }
    }
  }

  }  // warps without a score row

  tc::fence_before_sync();
  __syncthreads();
  if (s_abort && tid == 0) {
    atomicExch(p.status, kDevTimeout);
    atomicCAS(p.status + 1, 0, s_abort - 1 - (int)(tc::smem_u32(bars) & 0xffff));  // byte offset of the stuck barrier
  }
  if (warp == 0) tc::tmem_dealloc(tmem, kTmemCols);
}

// Failure-path probe: one warp waits, through the very wait the attention kernel uses, on an mbarrier that nothing
// ever completes.  The wait gives up after `limit` cycles, the kernel records the same status the attention kernel
// would (timeout + the barrier's offset) and returns normally: no trap, no endless loop, the context stays usable.
__global__ void bounded_wait_probe_kernel(int *status, long long limit) {
  __shared__ uint64_t never;
  __shared__ int s_abort;
  if (threadIdx.x == 0) {
    tc::mbar_init(&never, 1);
    tc::fence_barrier_init();
    s_abort = 0;
  }
  __syncthreads();
  volatile int *abortp = &s_abort;
  const bool ok = wait_or_abort(&never, 0, abortp, limit);
  __syncthreads();
  if (threadIdx.x == 0 && (!ok || s_abort)) {
    atomicExch(status, kDevTimeout);
    atomicCAS(status + 1, 0, s_abort - 1);
  }
}

}  // namespace

cudaError_t launch_bounded_wait_probe(int *status, long long limit_cycles, cudaStream_t st) {
  bounded_wait_probe_kernel<<<1, 32, 0, st>>>(status, limit_cycles);
  return cudaGetLastError();
}

cudaError_t launch_attention(const Params &p, __nv_bfloat16 *out, cudaStream_t st, int *launches) {
  // four softmax sets when their P images leave room for rings of at least 2 K and 3 V stages, else two
  SmemMap sm = make_smem_map(p, 4);
  int sets = 4;
  if (!sm.fits || sm.nv < 3) {
    sm = make_smem_map(p, 2);
    sets = 2;
  }
  if (!sm.fits) return cudaErrorInvalidConfiguration;
  cudaError_t e;
  const int grid = p.BH * ((p.Rt + 1) / 2);
  auto launch = [&](auto kernel, int nt) -> cudaError_t {
    cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm.total);
    if (err != cudaSuccess) return err;
    kernel<<<grid, nt, sm.total, st>>>(p, sm, out);
    return cudaSuccess;
  };
  const bool ordered = p.rank_scope != 0, fp4 = p.tier_active[0] != 0;
  auto pick = [&](auto dtag, auto stag) -> cudaError_t {
    constexpr int D = decltype(dtag)::value, S = decltype(stag)::value;
    constexpr int nt = Roles<S>::NT;
    return ordered ? (fp4 ? launch(attention_kernel<D, true, true, S>, nt) : launch(attention_kernel<D, true, false, S>, nt))
                   : (fp4 ? launch(attention_kernel<D, false, true, S>, nt) : launch(attention_kernel<D, false, false, S>, nt));
  };
  using I64 = std::integral_constant<int, 64>;
  using I128 = std::integral_constant<int, 128>;
  using S2 = std::integral_constant<int, 2>;
  using S4 = std::integral_constant<int, 4>;
  if (p.d == 128) e = sets == 4 ? pick(I128{}, S4{}) : pick(I128{}, S2{});
  else e = sets == 4 ? pick(I64{}, S4{}) : pick(I64{}, S2{});
  if (e != cudaSuccess) return e;
  *launches += 1;
  return cudaGetLastError();
}

}  // namespace da2

