// Kernel 2, second half: draft attention map, block-importance ranking and per-row block lists.
//   A = (1-lambda) softmax_row(logits_avg) + lambda softmax_row(logits_max)        (Def. 3.1, Eq. "v2-draft")
//   stable descending order of the scores, first quota -> 16-bit, next -> 8-bit, next -> 4-bit, rest skipped;
//   ties go to the lower index (Alg. 1, App. C.1).
// Output per query-block row: key-block ids grouped in execution order NVFP4 | INT8 | BF16 (Sec. 3.3 "Phased
// execution"), ascending inside a group, plus the three counts and the row's offset in its head's id array.
//
// Exact top-k without sorting: for each tier boundary a 4-pass radix select on the fp32 bit patterns (scores are
// non-negative, so bit patterns order like values) finds the boundary score and how many entries equal to it are
// still admitted; equal entries are admitted in index order through a prefix count.
//
// ROW scope: one CTA per (row, head) does everything.  HEAD scope (Alg. 1 as printed, one ranking over all R*R
// pairs of a head): the same steps split into small kernels with per-head histograms in the workspace.
#include "da2_internal.cuh"

namespace da2 {

namespace {

constexpr int NT = 256;

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ float block_max(float v, float *red) {
  v = warp_max(v);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  float r = red[0];
#pragma unroll
  for (int w = 1; w < NT / 32; ++w) r = fmaxf(r, red[w]);
  return r;
}
__device__ float block_sum(float v, float *red) {
  v = warp_sum(v);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  float r = 0.f;
#pragma unroll
  for (int w = 0; w < NT / 32; ++w) r += red[w];
  return r;
}

// Draft map row a of head bh into keys[] (fp32 bit patterns, shared memory) and into the global map.
__device__ void draft_map_row(const Params &p, int bh, int a, uint32_t *keys, float *red) {
  const float *l0 = p.logits[0] + ((size_t)bh * p.R + a) * p.R;
  const float *l1 = p.logits[1] + ((size_t)bh * p.R + a) * p.R;
  float *mp = p.map + ((size_t)bh * p.R + a) * p.R;
  float m0 = -INFINITY, m1 = -INFINITY;
  for (int i = threadIdx.x; i < p.R; i += NT) { m0 = fmaxf(m0, l0[i]); m1 = fmaxf(m1, l1[i]); }
  m0 = block_max(m0, red);
  m1 = block_max(m1, red);
  float z0 = 0.f, z1 = 0.f;
  for (int i = threadIdx.x; i < p.R; i += NT) { z0 += expf(l0[i] - m0); z1 += expf(l1[i] - m1); }
  z0 = block_sum(z0, red);
  z1 = block_sum(z1, red);
  const float w0 = 1.0f - p.lambda, w1 = p.lambda;
  for (int i = threadIdx.x; i < p.R; i += NT) {
    const float s = w0 * __fdiv_rn(expf(l0[i] - m0), z0) + w1 * __fdiv_rn(expf(l1[i] - m1), z1);
    keys[i] = __float_as_uint(s);
    mp[i] = s;
  }
  __syncthreads();
}

// One radix-select digit step on a 256-bin histogram (counts of the candidates' current digit), done by warp 0:
// finds the bin holding the need-th largest candidate.  out[0] = bin, out[1] = need minus the count above the bin.
__device__ void pick_bin(const uint32_t *hist, uint32_t need, uint32_t *out) {
  const int lane = threadIdx.x & 31;
  uint32_t c[8], local = 0;
#pragma unroll
  for (int i = 0; i < 8; ++i) { c[i] = hist[255 - (lane * 8 + i)]; local += c[i]; }
  uint32_t incl = local;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  uint32_t above = incl - local;  // candidates in higher bins than this lane's
  if (above < need && need <= incl) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      if (need <= above + c[i]) { out[0] = 255 - (lane * 8 + i); out[1] = need - above; break; }
      above += c[i];
    }
  }
}

// c-th largest of keys[0..n) (1 <= c <= n): value bits and how many entries equal to it are admitted.
__device__ void radix_select(const uint32_t *keys, int n, uint32_t c, uint32_t *hist, uint32_t *out,
                             uint32_t *value, uint32_t *take) {
  uint32_t prefix = 0, mask = 0, need = c;
  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int i = threadIdx.x; i < 256; i += NT) hist[i] = 0;
    __syncthreads();
    for (int i = threadIdx.x; i < n; i += NT) {
      const uint32_t key = keys[i];
      if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (threadIdx.x < 32) pick_bin(hist, need, out);
    __syncthreads();
    prefix |= out[0] << shift;
    mask |= 255u << shift;
    need = out[1];
    __syncthreads();
  }
  *value = prefix;
  *take = need;
}

// exclusive prefix over the block of NS counters per thread (thread order); totals returned to every thread
template <int NS>
__device__ void block_scan(int (&v)[NS], int (&total)[NS], int *scratch /* NS*NT */) {
  __syncthreads();
#pragma unroll
  for (int s = 0; s < NS; ++s) scratch[s * NT + threadIdx.x] = v[s];
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (warp < NS) {
    int *arr = scratch + warp * NT;
    int x[8], local = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) { x[i] = arr[lane * 8 + i]; local += x[i]; }
    int incl = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    int run = incl - local;
#pragma unroll
    for (int i = 0; i < 8; ++i) { arr[lane * 8 + i] = run; run += x[i]; }
    if (lane == 31) scratch[NS * NT + warp] = incl;
  }
  __syncthreads();
#pragma unroll
  for (int s = 0; s < NS; ++s) { v[s] = scratch[s * NT + threadIdx.x]; total[s] = scratch[NS * NT + s]; }
  __syncthreads();
}

struct Boundary { uint32_t value, take; };

__device__ __forceinline__ int tier_of(uint32_t key, const Boundary *bd, const int *eqrank) {
  // bd[0]: 16-bit boundary, bd[1]: 8-bit, bd[2]: 4-bit (cumulative).  Returns 2 (16-bit), 1, 0 or -1 (skip).
  if (key > bd[0].value || (key == bd[0].value && (uint32_t)eqrank[0] < bd[0].take)) return 2;
  if (key > bd[1].value || (key == bd[1].value && (uint32_t)eqrank[1] < bd[1].take)) return 1;
  if (key > bd[2].value || (key == bd[2].value && (uint32_t)eqrank[2] < bd[2].take)) return 0;
  return -1;
}

// ---------------------------------------------------------------------------------------------- ROW scope
__global__ void __launch_bounds__(NT) rank_row_kernel(Params p) {
  extern __shared__ uint32_t dyn[];
  uint32_t *keys = dyn;  // [R]
  __shared__ float red[NT / 32];
  __shared__ uint32_t hist[256];
  __shared__ uint32_t pick[2];
  __shared__ int scratch[3 * NT + 8];
  __shared__ Boundary bd[3];
  const int a = blockIdx.x, bh = blockIdx.y, R = p.R;

  draft_map_row(p, bh, a, keys, red);

  // cumulative boundaries: 16-bit, 16+8, 16+8+4
  long long cum = 0;
  for (int t = 0; t < 3; ++t) {
    const long long prev = cum;
    cum += p.quota[2 - t];
    uint32_t value, take;
    if (cum <= 0) { value = 0xffffffffu; take = 0; }
    else if (cum >= R) { value = 0u; take = (uint32_t)R; }
    else if (t > 0 && cum == prev) { value = bd[t - 1].value; take = bd[t - 1].take; }
    else radix_select(keys, R, (uint32_t)cum, hist, pick, &value, &take);
    __syncthreads();
    if (threadIdx.x == 0) { bd[t].value = value; bd[t].take = take; }
    __syncthreads();
  }

  // contiguous chunk per thread so that prefix counts follow index order
  const int per = (R + NT - 1) / NT;
  const int lo = min(R, (int)threadIdx.x * per), hi = min(R, lo + per);
  int eq[3] = {0, 0, 0}, tot[3];
  for (int i = lo; i < hi; ++i) {
    const uint32_t key = keys[i];
#pragma unroll
    for (int t = 0; t < 3; ++t) eq[t] += key == bd[t].value;
  }
  block_scan<3>(eq, tot, scratch);
  int cnt[3] = {0, 0, 0};
  {
    int er[3] = {eq[0], eq[1], eq[2]};
    for (int i = lo; i < hi; ++i) {
      const uint32_t key = keys[i];
      const int tr = tier_of(key, bd, er);
      if (tr >= 0) ++cnt[tr];
#pragma unroll
      for (int t = 0; t < 3; ++t) er[t] += key == bd[t].value;
    }
  }
  int pos[3] = {cnt[0], cnt[1], cnt[2]};
  block_scan<3>(pos, tot, scratch);
  const int stride = p.row_stride;
  uint16_t *ids = p.ids + (size_t)bh * p.ids_per_head + (size_t)a * stride;
  const int base[3] = {0, tot[0], tot[0] + tot[1]};
  {
    int er[3] = {eq[0], eq[1], eq[2]};
    for (int i = lo; i < hi; ++i) {
      const uint32_t key = keys[i];
      const int tr = tier_of(key, bd, er);
      if (tr >= 0) { ids[base[tr] + pos[tr]] = (uint16_t)i; ++pos[tr]; }
#pragma unroll
      for (int t = 0; t < 3; ++t) er[t] += key == bd[t].value;
    }
  }
  // prefix interactions lie outside the budget: every video row keeps all prefix blocks, in the 16-bit segment
  for (int j = threadIdx.x; j < p.Rp; j += NT) ids[tot[0] + tot[1] + tot[2] + j] = (uint16_t)(R + j);
  if (threadIdx.x == 0) {
    int *c = p.counts + ((size_t)bh * p.Rt + a) * 4;
    c[0] = tot[0]; c[1] = tot[1]; c[2] = tot[2] + p.Rp; c[3] = a * stride;
  }
}

// Prefix query rows are not sparse (App. C.1): their list is every block of the head, video and prefix, 16-bit.
__global__ void __launch_bounds__(NT) prefix_rows_kernel(Params p) {
  const int j = blockIdx.x, bh = blockIdx.y, a = p.R + j;
  const int pstride = (p.Rt + 7) / 8 * 8;
  const int off = p.R * p.row_stride + j * pstride;
  uint16_t *ids = p.ids + (size_t)bh * p.ids_per_head + off;
  for (int b = threadIdx.x; b < p.Rt; b += NT) ids[b] = (uint16_t)b;
  if (threadIdx.x == 0) {
    int *c = p.counts + ((size_t)bh * p.Rt + a) * 4;
    c[0] = 0; c[1] = 0; c[2] = p.Rt; c[3] = off;
  }
}

// --------------------------------------------------------------------------------------------- HEAD scope
// select scratch per head (uint32): [0..11]  (prefix, mask, need, pad) x 3 boundaries
//                                   [16..16+768) histograms 3 x 256
//                                   [1024..1024+3R) per-row equal counts -> exclusive prefixes
//                                   [1024+3R..1024+7R) per-row tier counts (3) + row total -> offsets
__device__ __forceinline__ uint32_t *sel_base(const Params &p, int bh) {
  return p.select + (size_t)bh * (4096 + 8 * (size_t)p.R);
}

__global__ void __launch_bounds__(NT) head_map_kernel(Params p) {
  extern __shared__ uint32_t dyn[];
  __shared__ float red[NT / 32];
  draft_map_row(p, blockIdx.y, blockIdx.x, dyn, red);
}

__global__ void head_init_kernel(Params p) {
  uint32_t *s = sel_base(p, blockIdx.x);
  const long long M = (long long)p.R * p.R;
  if (threadIdx.x < 3) {
    long long cum = 0;
    for (int t = 0; t <= (int)threadIdx.x; ++t) cum += p.quota[2 - t];
    uint32_t *b = s + threadIdx.x * 4;
    // b[3]: 0 = select normally, 1 = nothing admitted, 2 = everything admitted
    b[0] = 0; b[1] = 0; b[2] = (uint32_t)cum; b[3] = cum <= 0 ? 1u : (cum >= M ? 2u : 0u);
  }
  for (int i = threadIdx.x; i < 768; i += blockDim.x) s[16 + i] = 0;
}

__global__ void __launch_bounds__(NT) head_hist_kernel(Params p, int shift) {
  __shared__ uint32_t h[3][256];
  const int a = blockIdx.x, bh = blockIdx.y;
  uint32_t *s = sel_base(p, bh);
  for (int i = threadIdx.x; i < 768; i += NT) (&h[0][0])[i] = 0;
  __syncthreads();
  const uint32_t pf[3] = {s[0], s[4], s[8]}, mk[3] = {s[1], s[5], s[9]};
  const uint32_t *keys = reinterpret_cast<const uint32_t *>(p.map + ((size_t)bh * p.R + a) * p.R);
  for (int i = threadIdx.x; i < p.R; i += NT) {
    const uint32_t key = keys[i];
#pragma unroll
    for (int t = 0; t < 3; ++t)
      if ((key & mk[t]) == pf[t]) atomicAdd(&h[t][(key >> shift) & 255u], 1u);
  }
  __syncthreads();
  for (int i = threadIdx.x; i < 768; i += NT) {
    const uint32_t c = (&h[0][0])[i];
    if (c) atomicAdd(&s[16 + i], c);
  }
}

__global__ void head_pick_kernel(Params p, int shift) {
  __shared__ uint32_t out[3][2];
  uint32_t *s = sel_base(p, blockIdx.x);
  const int t = threadIdx.x >> 5;  // 3 warps, one per boundary
  if (t < 3) {
    if (s[t * 4 + 3] == 0) pick_bin(s + 16 + t * 256, s[t * 4 + 2], out[t]);
  }
  __syncthreads();
  if (threadIdx.x < 3 && s[threadIdx.x * 4 + 3] == 0) {
    uint32_t *b = s + threadIdx.x * 4;
    b[0] |= out[threadIdx.x][0] << shift;
    b[1] |= 255u << shift;
    b[2] = out[threadIdx.x][1];
  }
  __syncthreads();
  for (int i = threadIdx.x; i < 768; i += blockDim.x) s[16 + i] = 0;
}

__device__ __forceinline__ void load_boundaries(const uint32_t *s, int R, Boundary *bd) {
  for (int t = 0; t < 3; ++t) {
    const uint32_t mode = s[t * 4 + 3];
    if (mode == 1) { bd[t].value = 0xffffffffu; bd[t].take = 0; }
    else if (mode == 2) { bd[t].value = 0u; bd[t].take = 0xffffffffu; }
    else { bd[t].value = s[t * 4]; bd[t].take = s[t * 4 + 2]; }
  }
  (void)R;
}

// per-row counts of entries equal to each boundary score
__global__ void __launch_bounds__(NT) head_eqcount_kernel(Params p) {
  __shared__ int scratch[3 * NT + 8];
  const int a = blockIdx.x, bh = blockIdx.y;
  uint32_t *s = sel_base(p, bh);
  Boundary bd[3];
  load_boundaries(s, p.R, bd);
  const uint32_t *keys = reinterpret_cast<const uint32_t *>(p.map + ((size_t)bh * p.R + a) * p.R);
  int eq[3] = {0, 0, 0}, tot[3];
  for (int i = threadIdx.x; i < p.R; i += NT) {
    const uint32_t key = keys[i];
#pragma unroll
    for (int t = 0; t < 3; ++t) eq[t] += key == bd[t].value;
  }
  block_scan<3>(eq, tot, scratch);
  if (threadIdx.x < 3) s[1024 + threadIdx.x * p.R + a] = (uint32_t)tot[threadIdx.x];
}

// exclusive prefix over rows of `narr` arrays of length R stored back to back at s[base...]; totals dropped
__global__ void __launch_bounds__(NT) head_rowscan_kernel(Params p, int base_words, int narr) {
  __shared__ int scratch[1 * NT + 8];
  uint32_t *s = sel_base(p, blockIdx.x) + base_words;
  const int per = (p.R + NT - 1) / NT;
  for (int arr = 0; arr < narr; ++arr) {
    uint32_t *x = s + (size_t)arr * p.R;
    const int lo = min(p.R, (int)threadIdx.x * per), hi = min(p.R, lo + per);
    int v[1] = {0}, tot[1];
    for (int i = lo; i < hi; ++i) v[0] += (int)x[i];
    block_scan<1>(v, tot, scratch);
    int run = v[0];
    for (int i = lo; i < hi; ++i) { const int c = (int)x[i]; x[i] = (uint32_t)run; run += c; }
    __syncthreads();
  }
}

// mode 0: count the row's entries per tier; mode 1: emit ids at the row's offset
__global__ void __launch_bounds__(NT) head_emit_kernel(Params p, int mode) {
  extern __shared__ uint32_t dyn[];
  uint32_t *keys = dyn;
  __shared__ int scratch[3 * NT + 8];
  const int a = blockIdx.x, bh = blockIdx.y, R = p.R;
  uint32_t *s = sel_base(p, bh);
  Boundary bd[3];
  load_boundaries(s, R, bd);
  const uint32_t *gk = reinterpret_cast<const uint32_t *>(p.map + ((size_t)bh * R + a) * R);
  for (int i = threadIdx.x; i < R; i += NT) keys[i] = gk[i];
  __syncthreads();
  const int per = (R + NT - 1) / NT;
  const int lo = min(R, (int)threadIdx.x * per), hi = min(R, lo + per);
  int eq[3] = {0, 0, 0}, tot[3];
  for (int i = lo; i < hi; ++i) {
#pragma unroll
    for (int t = 0; t < 3; ++t) eq[t] += keys[i] == bd[t].value;
  }
  block_scan<3>(eq, tot, scratch);
#pragma unroll
  for (int t = 0; t < 3; ++t) eq[t] += (int)s[1024 + t * R + a];  // equal entries in earlier rows of the head
  int cnt[3] = {0, 0, 0};
  {
    int er[3] = {eq[0], eq[1], eq[2]};
    for (int i = lo; i < hi; ++i) {
      const int tr = tier_of(keys[i], bd, er);
      if (tr >= 0) ++cnt[tr];
#pragma unroll
      for (int t = 0; t < 3; ++t) er[t] += keys[i] == bd[t].value;
    }
  }
  int pos[3] = {cnt[0], cnt[1], cnt[2]};
  block_scan<3>(pos, tot, scratch);
  uint32_t *rowtot = s + 1024 + 3 * R;  // [R] totals -> offsets after the row scan
  if (mode == 0) {
    if (threadIdx.x == 0) {
      int *c = p.counts + ((size_t)bh * R + a) * 4;
      c[0] = tot[0]; c[1] = tot[1]; c[2] = tot[2];
      rowtot[a] = (uint32_t)(tot[0] + tot[1] + tot[2]);
    }
    return;
  }
  const uint32_t off = rowtot[a];
  uint16_t *ids = p.ids + (size_t)bh * p.ids_per_head + off;
  const int base[3] = {0, tot[0], tot[0] + tot[1]};
  int er[3] = {eq[0], eq[1], eq[2]};
  for (int i = lo; i < hi; ++i) {
    const int tr = tier_of(keys[i], bd, er);
    if (tr >= 0) { ids[base[tr] + pos[tr]] = (uint16_t)i; ++pos[tr]; }
#pragma unroll
    for (int t = 0; t < 3; ++t) er[t] += keys[i] == bd[t].value;
  }
  if (threadIdx.x == 0) p.counts[((size_t)bh * R + a) * 4 + 3] = (int)off;
}

}  // namespace

// Draft map rows only (softmax of both logit branches and their mixture into p.map); used by callers that want
// the map without the ranking.
cudaError_t launch_map_rows(const Params &p, cudaStream_t st, int *launches) {
  dim3 grid(p.R, p.BH);
  const size_t smem = (size_t)p.R * sizeof(uint32_t);
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(head_map_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  head_map_kernel<<<grid, NT, smem, st>>>(p);
  *launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_rank(const Params &p, cudaStream_t st, int *launches) {
  dim3 grid(p.R, p.BH);
  const size_t smem = (size_t)p.R * sizeof(uint32_t);
  cudaError_t e;
  if (p.rank_scope == DA2_RANK_ROW) {
    if (smem > 48 * 1024) {
      e = cudaFuncSetAttribute(rank_row_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
    }
    rank_row_kernel<<<grid, NT, smem, st>>>(p);
    *launches += 1;
    return cudaGetLastError();
  }
  if (smem > 48 * 1024) {
    e = cudaFuncSetAttribute(head_map_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(head_emit_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  head_map_kernel<<<grid, NT, smem, st>>>(p);
  head_init_kernel<<<p.BH, NT, 0, st>>>(p);
  *launches += 2;
  for (int shift = 24; shift >= 0; shift -= 8) {
    head_hist_kernel<<<grid, NT, 0, st>>>(p, shift);
    head_pick_kernel<<<p.BH, 96, 0, st>>>(p, shift);
    *launches += 2;
  }
  head_eqcount_kernel<<<grid, NT, 0, st>>>(p);
  head_rowscan_kernel<<<p.BH, NT, 0, st>>>(p, 1024, 3);
  head_emit_kernel<<<grid, NT, smem, st>>>(p, 0);
  head_rowscan_kernel<<<p.BH, NT, 0, st>>>(p, 1024 + 3 * p.R, 1);
  head_emit_kernel<<<grid, NT, smem, st>>>(p, 1);
  *launches += 5;
  return cudaGetLastError();
}


// Scheduling order of the query blocks of a head for the attention kernel: by decreasing list length, ties by index.
// O(R^2) comparisons per head on lengths staged in shared memory (R is a few thousand at most).
namespace {
__global__ void __launch_bounds__(256) order_rows_kernel(Params p) {
  extern __shared__ int s_len[];
  const int bh = blockIdx.x, R = p.R, Rp = 2 * ((R + 1) / 2);
  const int *cnt = p.counts + (size_t)bh * R * 4;
  for (int a = threadIdx.x; a < R; a += blockDim.x) s_len[a] = cnt[a * 4] + cnt[a * 4 + 1] + cnt[a * 4 + 2];
  __syncthreads();
  uint16_t *ord = p.order + (size_t)bh * Rp;
  if (threadIdx.x == 0 && Rp > R) ord[R] = 0xFFFFu;
  for (int a = threadIdx.x; a < R; a += blockDim.x) {
    const int la = s_len[a];
    int pos = 0;
    for (int b = 0; b < R; ++b) {
      const int lb = s_len[b];
      pos += (lb > la) || (lb == la && b < a);
    }
    ord[pos] = (uint16_t)a;
  }
}
}  // namespace

cudaError_t launch_prefix_rows(const Params &p, cudaStream_t st, int *launches) {
  if (p.Rp == 0) return cudaSuccess;
  prefix_rows_kernel<<<dim3(p.Rp, p.BH), NT, 0, st>>>(p);
  *launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_order(const Params &p, cudaStream_t st, int *launches) {
  const size_t smem = (size_t)p.R * sizeof(int);
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(order_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  order_rows_kernel<<<p.BH, 256, smem, st>>>(p);
  *launches += 1;
  return cudaGetLastError();
}

}  // namespace da2
