// C-ABI entry points of the da2 library: host-side plan (tiling, quotas, workspace layout) and the two device calls.
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>
#include <map>
#include <mutex>
#include <tuple>
#include <vector>

#include "da2_internal.cuh"

namespace {

inline uint64_t align_up(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }

struct Carver {
  uint64_t cur = 0;
  uint64_t take(uint64_t bytes) {
    uint64_t off = cur;
    cur = align_up(cur + bytes, 256);
    return off;
  }
};

// Integer quotas from fractions of M candidates (App. C.1: integer quotas T_p whose sum is the retained budget).
// Cumulative round-half-up keeps the three counts consistent with the rounded total.
void quotas_from_fractions(double f16, double f8, double f4, long long M, long long out[3]) {
  long long c16 = (long long)std::floor(f16 * (double)M + 0.5);
  long long c8 = (long long)std::floor((f16 + f8) * (double)M + 0.5);
  long long c4 = (long long)std::floor((f16 + f8 + f4) * (double)M + 0.5);
  c16 = c16 > M ? M : c16;
  c8 = c8 > M ? M : c8;
  c4 = c4 > M ? M : c4;
  out[2] = c16;
  out[1] = c8 - c16;
  out[0] = c4 - c8;
}

da2::Params make_params(const da2_plan_t *plan, void *workspace) {
  const da2_plan_info_t &I = plan->info;
  da2::Params p;
  std::memset(&p, 0, sizeof(p));
  p.B = I.B; p.H = I.H; p.T = I.T; p.Hg = I.Hg; p.Wg = I.Wg; p.d = I.head_dim;
  p.nty = I.nty; p.ntx = I.ntx; p.R_f = I.R_f; p.R = I.R; p.N = I.N; p.BH = I.B * I.H;
  p.P = I.n_prefix; p.Rp = I.R_prefix; p.Rt = I.R + I.R_prefix; p.Ntot = I.N + I.n_prefix;
  p.row_stride = I.row_stride;
  p.part = I.partition; p.part_tr = I.part_transposed; p.part_bands = I.part_bands; p.part_n = I.part_n;
  p.part_rem = I.part_rem;
  p.rank_scope = I.rank_scope;
  for (int t = 0; t < 3; ++t) {
    p.tier_active[t] = I.tier_active[t];
    p.quota[t] = I.quota[t];
    p.qrec_bytes[t] = I.qrec_bytes[t];
    p.kvrec_bytes[t] = I.kvrec_bytes[t];
  }
  p.ids_per_head = I.ids_per_head;
  p.lambda = I.lambda;
  p.scale = I.softmax_scale;
  uint8_t *w = (uint8_t *)workspace;
  p.status = (int *)(w + I.off_status);
  p.amax = (uint32_t *)(w + I.off_amax);
  p.vmax = (uint32_t *)(w + I.off_vmax);
  p.gscale = (float *)(w + I.off_gscale);
  for (int i = 0; i < 4; ++i) p.desc[i] = (float *)(w + I.off_desc[i]);
  for (int i = 0; i < 2; ++i) p.logits[i] = (float *)(w + I.off_logits[i]);
  p.map = (float *)(w + I.off_map);
  p.counts = (int *)(w + I.off_counts);
  p.ids = (uint16_t *)(w + I.off_ids);
  p.select = (uint32_t *)(w + I.off_select);
  p.order = (uint16_t *)(w + I.off_order);
  for (int t = 0; t < 3; ++t) {
    p.qrec[t] = w + I.off_qrec[t];
    p.kvrec[t] = w + I.off_kvrec[t];
  }
  p.dq8 = (float *)(w + I.off_dq8);
  p.dk8 = (float *)(w + I.off_dk8);
  p.dv8 = (float *)(w + I.off_dv8);
  p.region_cell = (int *)(w + plan->off_region_cell);
  p.region_mask = (unsigned long long *)(w + plan->off_region_mask);
  return p;
}

bool misaligned(const void *ptr, uintptr_t a) { return ((uintptr_t)ptr % a) != 0; }

// Balanced ragged partition of one H x W frame into Rf regions (App. C.2): candidates are band orders (see
// slot_token in da2_internal.cuh) cut into Rf runs of n or n + 1 cells; a candidate counts if every run is
// 4-connected, and the one with the fewest cut edges (smallest total perimeter, Eq. "region-perimeter") wins; ties go
// to bands along rows, then to fewer bands.  Host only, integer work, once per plan.
struct BandChoice { int transposed, bands; long long perimeter; };

int band_cell(int H, int W, int bands, int transposed, int pos) {
  const int L = transposed ? W : H, M = transposed ? H : W;
  const int hb = L / bands, extra = L % bands, big = extra * (hb + 1) * M;
  int b, h, q;
  if (pos < big) { h = hb + 1; b = pos / (h * M); q = pos - b * h * M; }
  else { h = hb; pos -= big; b = pos / (h * M); q = pos - b * h * M; b += extra; }
  const int l0 = b * hb + (b < extra ? b : extra);
  const int i = q / h, k = q - i * h;
  const int m = (b & 1) ? M - 1 - i : i;
  const int l = l0 + ((i & 1) ? h - 1 - k : k);
  return transposed ? m * W + l : l * W + m;
}

BandChoice choose_bands(int H, int W, int Rf) {
  const int HW = H * W, n = HW / Rf, rem = HW % Rf;
  std::vector<int> region(HW), parent(HW);
  BandChoice best = {0, 0, -1};
  for (int tr = 0; tr < 2; ++tr)
    for (int bands = 1; bands <= (tr ? W : H); ++bands) {
      int pos = 0;
      for (int a = 0; a < Rf; ++a)
        for (int j = 0; j < n + (a < rem); ++j) region[band_cell(H, W, bands, tr, pos++)] = a;
      // union-find over equal-region neighbours; the cut edges are counted on the way
      for (int c = 0; c < HW; ++c) parent[c] = c;
      auto find = [&](int c) { while (parent[c] != c) { parent[c] = parent[parent[c]]; c = parent[c]; } return c; };
      long long cut = 0;
      int comps = HW;
      for (int y = 0; y < H; ++y)
        for (int x = 0; x < W; ++x) {
          const int c = y * W + x;
          const int nb[2] = {x + 1 < W ? c + 1 : -1, y + 1 < H ? c + W : -1};
          for (int e = 0; e < 2; ++e) {
            if (nb[e] < 0) continue;
            if (region[nb[e]] != region[c]) { ++cut; continue; }
            const int ra = find(c), rb = find(nb[e]);
            if (ra != rb) { parent[ra] = rb; --comps; }
          }
        }
      if (comps != Rf) continue;
      const long long per = 2ll * (H + W) + 2 * cut;
      if (best.perimeter < 0 || per < best.perimeter) best = {tr, bands, per};
    }
  return best;
}

// The search costs a few milliseconds and depends on the frame's grid only: plans of the same grid (the per-group plans
// of the host entry, for one) share its result.
BandChoice cached_bands(int H, int W, int Rf) {
  static std::mutex mu;
  static std::map<std::tuple<int, int, int>, BandChoice> memo;
  const auto key = std::make_tuple(H, W, Rf);
  {
    std::lock_guard<std::mutex> lock(mu);
    auto it = memo.find(key);
    if (it != memo.end()) return it->second;
  }
  const BandChoice ch = choose_bands(H, W, Rf);
  std::lock_guard<std::mutex> lock(mu);
  memo.emplace(key, ch);
  return ch;
}

// kernels enqueued by the calling thread's last da2_prepare / da2_refresh_operands / da2_attention_fwd
thread_local int t_last_launches = 0;

// Caller-fixed NVFP4 per-tensor scales travel as kernel arguments (copied when the launch is enqueued, so the call
// stays legal inside a stream capture; a copy from pageable host memory would not be).
constexpr int kScaleChunk = 256;
struct ScaleChunk { float v[kScaleChunk]; };
__global__ void set_gscale_kernel(float *gscale, int which, int first, int n, ScaleChunk c) {
  const int i = threadIdx.x;
  if (i < n) gscale[(size_t)(first + i) * 4 + which] = c.v[i];
}

}  // namespace

extern "C" {

da2_status_t da2_plan(const da2_config_t *cfg, da2_plan_t **plan_out) {
  if (!cfg || !plan_out) return DA2_ERR_INVALID_ARG;
  *plan_out = nullptr;
  if (cfg->B < 1 || cfg->H < 1 || cfg->T < 1 || cfg->Hg < 1 || cfg->Wg < 1) return DA2_ERR_INVALID_ARG;
  if ((long long)cfg->B * cfg->H > 32767) return DA2_ERR_UNSUPPORTED;  // heads index grid dimensions y and z
  if (cfg->frac16 < 0 || cfg->frac8 < 0 || cfg->frac4 < 0 || cfg->frac16 + cfg->frac8 + cfg->frac4 > 1.0 + 1e-12)
    return DA2_ERR_INVALID_ARG;
  if (!(cfg->lambda >= 0.0f && cfg->lambda <= 1.0f)) return DA2_ERR_INVALID_ARG;
  if (cfg->rank_scope != DA2_RANK_ROW && cfg->rank_scope != DA2_RANK_HEAD) return DA2_ERR_INVALID_ARG;
  if (cfg->n_prefix < 0 || cfg->n_prefix > (1 << 20)) return DA2_ERR_INVALID_ARG;
  // prefix rows need a list layout with per-row offsets that the head-level ranking does not reserve room for
  if (cfg->n_prefix > 0 && cfg->rank_scope == DA2_RANK_HEAD) return DA2_ERR_UNSUPPORTED;
  if (cfg->head_dim != 64 && cfg->head_dim != 128) return DA2_ERR_UNSUPPORTED;
  if (cfg->tile_h != 8 || cfg->tile_w != 8) return DA2_ERR_UNSUPPORTED;
  if (cfg->partition != DA2_PARTITION_TILES && cfg->partition != DA2_PARTITION_BALANCED) return DA2_ERR_INVALID_ARG;
  // the balanced partition packs regions into blocks of the kernels' 64 slots; 128-token blocks are not built
  if (cfg->partition == DA2_PARTITION_BALANCED && cfg->capacity != da2::kSlots) return DA2_ERR_UNSUPPORTED;

  da2_plan_t *plan = new (std::nothrow) da2_plan_t();
  if (!plan) return DA2_ERR_INTERNAL;
  plan->cfg = *cfg;
  for (int i = 0; i < 3; ++i) plan->g_host[i] = nullptr;

  da2_plan_info_t &I = plan->info;
  std::memset(&I, 0, sizeof(I));
  I.B = cfg->B; I.H = cfg->H; I.T = cfg->T; I.Hg = cfg->Hg; I.Wg = cfg->Wg; I.head_dim = cfg->head_dim;
  I.tile_h = 8; I.tile_w = 8;
  I.nty = (cfg->Hg + 7) / 8;
  I.ntx = (cfg->Wg + 7) / 8;
  I.R_f = I.nty * I.ntx;
  I.partition = cfg->partition;
  if (cfg->partition == DA2_PARTITION_BALANCED) {
    const int HW = cfg->Hg * cfg->Wg;
    I.R_f = (HW + da2::kSlots - 1) / da2::kSlots;
    const BandChoice ch = cached_bands(cfg->Hg, cfg->Wg, I.R_f);
    I.part_transposed = ch.transposed;
    I.part_bands = ch.bands;
    I.part_perimeter = ch.perimeter;
    I.part_n = HW / I.R_f;
    I.part_rem = HW % I.R_f;
  }
  long long R = (long long)cfg->T * I.R_f;
  if (R > 16384) { delete plan; return DA2_ERR_UNSUPPORTED; }  // ids are uint16; row buffers live in shared memory
  const long long Rp = ((long long)cfg->n_prefix + da2::kSlots - 1) / da2::kSlots, Rt = R + Rp;
  if (Rt > 65535) { delete plan; return DA2_ERR_UNSUPPORTED; }
  I.n_prefix = cfg->n_prefix;
  I.R_prefix = (int32_t)Rp;
  I.R = (int32_t)R;
  I.S = da2::kSlots;
  I.N = (int64_t)cfg->T * cfg->Hg * cfg->Wg;
  I.rank_scope = cfg->rank_scope;
  I.lambda = cfg->lambda;
  I.softmax_scale = cfg->softmax_scale > 0.0f ? cfg->softmax_scale : 1.0f / std::sqrt((float)cfg->head_dim);
  const long long M = cfg->rank_scope == DA2_RANK_ROW ? R : R * R;
  long long qt[3];
  quotas_from_fractions(cfg->frac16, cfg->frac8, cfg->frac4, M, qt);
  for (int t = 0; t < 3; ++t) { I.quota[t] = qt[t]; I.tier_active[t] = qt[t] > 0; }
  if (Rp > 0) I.tier_active[2] = 1;  // prefix interactions run in the 16-bit tier, outside the budget

  const uint64_t BH = (uint64_t)cfg->B * cfg->H, d = cfg->head_dim, S = da2::kSlots;
  const long long kept = qt[0] + qt[1] + qt[2];
  if (cfg->rank_scope == DA2_RANK_ROW) {
    long long stride = (kept + Rp + 7) / 8 * 8;
    if (stride == 0) stride = 8;
    I.row_stride = (int32_t)stride;
    I.ids_per_head = stride * R + Rp * ((Rt + 7) / 8 * 8);  // video rows, then the prefix rows (every block each)
  } else {
    I.row_stride = 0;
    I.ids_per_head = (kept + 7) / 8 * 8 + 8;
  }

  // record sizes: tier 0 NVFP4, tier 1 INT8/E4M3, tier 2 BF16
  I.qrec_bytes[0] = (uint32_t)(S * d / 2 + (d / 64) * da2::kSfAtomBytes);
  I.qrec_bytes[1] = (uint32_t)(S * d);
  I.qrec_bytes[2] = (uint32_t)(S * d * 2);
  I.kvrec_bytes[0] = (uint32_t)(S * d / 2 + (d / 64) * da2::kSfAtomBytes + d * S / 2 + da2::kSfAtomBytes);
  I.kvrec_bytes[1] = (uint32_t)(2 * S * d);
  I.kvrec_bytes[2] = (uint32_t)(4 * S * d);

  Carver c;
  I.off_status = c.take(64 * 4);
  I.off_amax = c.take(BH * 4 * 4);
  I.off_vmax = c.take(BH * d * 4);
  I.off_gscale = c.take(BH * 4 * 4);
  for (int i = 0; i < 4; ++i) I.off_desc[i] = c.take(BH * R * d * 4);
  for (int i = 0; i < 2; ++i) I.off_logits[i] = c.take(BH * R * R * 4);
  I.off_map = c.take(BH * R * R * 4);
  I.off_counts = c.take(BH * (uint64_t)Rt * 4 * 4);
  I.off_ids = c.take(BH * (uint64_t)I.ids_per_head * 2);
  I.off_select = c.take(BH * (4096 + 8 * (uint64_t)R) * 4);
  for (int t = 0; t < 3; ++t) {
    const uint64_t blocks = t == 2 ? (uint64_t)Rt : (uint64_t)R;  // the 16-bit tier also holds the prefix blocks
    I.off_qrec[t] = c.take(I.tier_active[t] ? BH * blocks * I.qrec_bytes[t] : 0);
    I.off_kvrec[t] = c.take(I.tier_active[t] ? BH * blocks * I.kvrec_bytes[t] : 0);
  }
  I.off_dq8 = c.take(BH * R * 4);
  I.off_dk8 = c.take(BH * R * 4);
  I.off_dv8 = c.take(BH * d * 4);
  I.off_order = c.take(BH * (uint64_t)(2 * ((R + 1) / 2)) * 2);
  plan->off_region_cell = c.take((uint64_t)I.R_f * da2::kSlots * 4);
  plan->off_region_mask = c.take((uint64_t)I.R_f * 8);
  I.workspace_bytes = c.cur;

  const float *src[3] = {cfg->g_q, cfg->g_k, cfg->g_v};
  for (int i = 0; i < 3; ++i) {
    if (!src[i]) continue;
    plan->g_host[i] = (float *)std::malloc(BH * sizeof(float));
    if (!plan->g_host[i]) { da2_plan_destroy(plan); return DA2_ERR_INTERNAL; }
    for (uint64_t j = 0; j < BH; ++j) {
      if (!(src[i][j] > 0.0f)) { da2_plan_destroy(plan); return DA2_ERR_INVALID_ARG; }
      plan->g_host[i][j] = src[i][j];
    }
  }
  plan->cfg.g_q = plan->g_host[0];
  plan->cfg.g_k = plan->g_host[1];
  plan->cfg.g_v = plan->g_host[2];
  *plan_out = plan;
  return DA2_OK;
}

da2_status_t da2_plan_info(const da2_plan_t *plan, da2_plan_info_t *info) {
  if (!plan || !info) return DA2_ERR_INVALID_ARG;
  *info = plan->info;
  return DA2_OK;
}

namespace {

// da2_prepare and da2_refresh_operands: the same pipeline with or without the selection stages
da2_status_t prepare_impl(const da2_plan_t *plan, const void *q, const void *k, const void *v, void *workspace,
                          size_t workspace_bytes, void *stream, bool select) {
  if (!plan || !q || !k || !v || !workspace) return DA2_ERR_INVALID_ARG;
  if (misaligned(q, 16) || misaligned(k, 16) || misaligned(v, 16) || misaligned(workspace, 256))
    return DA2_ERR_INVALID_ARG;
  if (workspace_bytes < plan->info.workspace_bytes) return DA2_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = (cudaStream_t)stream;
  da2::Params p = make_params(plan, workspace);
  const da2_plan_info_t &I = plan->info;
  int launches = 0;
  t_last_launches = 0;
  // status word, head maxima and per-channel maxima start at zero (they are contiguous)
  if (cudaMemsetAsync((uint8_t *)workspace + I.off_status, 0, I.off_gscale - I.off_status, st) != cudaSuccess)
    return DA2_ERR_CUDA;
  const __nv_bfloat16 *qb = (const __nv_bfloat16 *)q, *kb = (const __nv_bfloat16 *)k, *vb = (const __nv_bfloat16 *)v;
  if (da2::launch_pool(p, qb, kb, vb, st, &launches) != cudaSuccess) return DA2_ERR_CUDA;
  for (int i = 0; i < 3; ++i) {  // caller-fixed NVFP4 per-tensor scales replace the derived ones
    if (!plan->g_host[i]) continue;
    for (int first = 0; first < p.BH; first += kScaleChunk) {
      ScaleChunk c;
      const int n = p.BH - first < kScaleChunk ? p.BH - first : kScaleChunk;
      std::memcpy(c.v, plan->g_host[i] + first, sizeof(float) * (size_t)n);
      set_gscale_kernel<<<1, kScaleChunk, 0, st>>>(p.gscale, i, first, n, c);
      if (cudaGetLastError() != cudaSuccess) return DA2_ERR_CUDA;
      launches += 1;
    }
  }
  if (select) {
    if (da2::launch_draft(p, st, &launches) != cudaSuccess) return DA2_ERR_CUDA;
    if (da2::launch_rank(p, st, &launches) != cudaSuccess) return DA2_ERR_CUDA;
    if (da2::launch_prefix_rows(p, st, &launches) != cudaSuccess) return DA2_ERR_CUDA;
    // rows of unequal length (HEAD scope) are paired by length; with per-row budgets the order is the identity
    if (plan->info.rank_scope != 0 && da2::launch_order(p, st, &launches) != cudaSuccess) return DA2_ERR_CUDA;
  }
  if (da2::launch_prep(p, qb, kb, vb, st, &launches) != cudaSuccess) return DA2_ERR_CUDA;
  t_last_launches = launches;
  return DA2_OK;
}

}  // namespace

da2_status_t da2_prepare(const da2_plan_t *plan, const void *q, const void *k, const void *v, void *workspace,
                         size_t workspace_bytes, void *stream) {
  return prepare_impl(plan, q, k, v, workspace, workspace_bytes, stream, true);
}

da2_status_t da2_refresh_operands(const da2_plan_t *plan, const void *q, const void *k, const void *v,
                                  void *workspace, size_t workspace_bytes, void *stream) {
  return prepare_impl(plan, q, k, v, workspace, workspace_bytes, stream, false);
}

da2_status_t da2_prepare_cached_scales(const da2_plan_t *plan, const void *q, const void *k, const void *v,
                                       void *workspace, size_t workspace_bytes, int32_t reselect, void *stream) {
  if (!plan || !q || !k || !v || !workspace) return DA2_ERR_INVALID_ARG;
  if (misaligned(q, 16) || misaligned(k, 16) || misaligned(v, 16) || misaligned(workspace, 256))
    return DA2_ERR_INVALID_ARG;
  if (workspace_bytes < plan->info.workspace_bytes) return DA2_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = (cudaStream_t)stream;
  da2::Params p = make_params(plan, workspace);
  int launches = 0;
  t_last_launches = 0;
  // only the status word is cleared: the statistics and the scales derived from them stay as the earlier call left them
  if (cudaMemsetAsync((uint8_t *)workspace + plan->info.off_status, 0, 64 * sizeof(int), st) != cudaSuccess)
    return DA2_ERR_CUDA;
  const __nv_bfloat16 *qb = (const __nv_bfloat16 *)q, *kb = (const __nv_bfloat16 *)k, *vb = (const __nv_bfloat16 *)v;
  if (da2::launch_prep(p, qb, kb, vb, st, &launches, /*pool=*/true) != cudaSuccess) return DA2_ERR_CUDA;
  if (reselect) {
    if (da2::launch_draft(p, st, &launches) != cudaSuccess) return DA2_ERR_CUDA;
    if (da2::launch_rank(p, st, &launches) != cudaSuccess) return DA2_ERR_CUDA;
    if (da2::launch_prefix_rows(p, st, &launches) != cudaSuccess) return DA2_ERR_CUDA;
    if (plan->info.rank_scope != 0 && da2::launch_order(p, st, &launches) != cudaSuccess) return DA2_ERR_CUDA;
  }
  t_last_launches = launches;
  return DA2_OK;
}

da2_status_t da2_attention_fwd(const da2_plan_t *plan, const void *q, const void *k, const void *v,
                               const void *workspace, void *out, void *stream) {
  if (!plan || !q || !k || !v || !workspace || !out) return DA2_ERR_INVALID_ARG;
  if (misaligned(out, 16) || misaligned(workspace, 256)) return DA2_ERR_INVALID_ARG;
  if (out == q || out == k || out == v) return DA2_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  da2::Params p = make_params(plan, const_cast<void *>(workspace));
  int launches = 0;
  t_last_launches = 0;
  if (da2::launch_attention(p, (__nv_bfloat16 *)out, st, &launches) != cudaSuccess) return DA2_ERR_CUDA;
  t_last_launches = launches;
  return DA2_OK;
}

da2_status_t da2_selfcheck_quantiser_arithmetic(int32_t mode, int32_t n_divisors, uint32_t seed, void *out_dev,
                                                void *stream) {
  if (!out_dev || mode < 0 || mode > 2 || misaligned(out_dev, 8)) return DA2_ERR_INVALID_ARG;
  if (mode != 2 && (n_divisors < 1 || n_divisors > (1 << 22))) return DA2_ERR_INVALID_ARG;
  if (da2::launch_quantiser_selfcheck(mode, n_divisors, seed, (unsigned long long *)out_dev, (cudaStream_t)stream) !=
      cudaSuccess)
    return DA2_ERR_CUDA;
  return DA2_OK;
}

da2_status_t da2_device_status(const da2_plan_t *plan, const void *workspace, void *stream) {
  if (!plan || !workspace) return DA2_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  int word[4] = {0, 0, 0, 0};
  if (cudaMemcpyAsync(word, (const uint8_t *)workspace + plan->info.off_status, sizeof(word),
                      cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return DA2_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return DA2_ERR_CUDA;
  if (word[0] == da2::kDevOk) return DA2_OK;
  if (word[0] == da2::kDevTimeout) return DA2_ERR_TIMEOUT;
  return DA2_ERR_INTERNAL;
}

int64_t da2_plan_slot_token(const da2_plan_t *plan, int32_t block, int32_t slot) {
  if (!plan || block < 0 || block >= plan->info.R + plan->info.R_prefix || slot < 0 || slot >= da2::kSlots) return -2;
  const da2::Params p = make_params(plan, nullptr);
  if (!((da2::block_valid_mask(p, block) >> slot) & 1ull)) return -1;
  return (int64_t)da2::slot_token(p, block, slot);
}

int32_t da2_last_launch_count(const da2_plan_t *plan) { return plan ? t_last_launches : 0; }

da2_status_t da2_probe_bounded_wait(const da2_plan_t *plan, void *workspace, int64_t limit_cycles, void *stream) {
  if (!plan || !workspace || limit_cycles < 1 || limit_cycles > 2000000000ll) return DA2_ERR_INVALID_ARG;
  if (misaligned(workspace, 256)) return DA2_ERR_INVALID_ARG;
  int *status = (int *)((uint8_t *)workspace + plan->info.off_status);
  if (da2::launch_bounded_wait_probe(status, (long long)limit_cycles, (cudaStream_t)stream) != cudaSuccess)
    return DA2_ERR_CUDA;
  return DA2_OK;
}

void da2_plan_destroy(da2_plan_t *plan) {
  if (!plan) return;
  for (int i = 0; i < 3; ++i) std::free(plan->g_host[i]);
  delete plan;
}

const char *da2_status_string(da2_status_t status) {
  switch (status) {
    case DA2_OK: return "ok";
    case DA2_ERR_INVALID_ARG: return "invalid argument";
    case DA2_ERR_UNSUPPORTED: return "unsupported configuration";
    case DA2_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case DA2_ERR_CUDA: return "CUDA error";
    case DA2_ERR_TIMEOUT: return "device-side wait timed out";
    case DA2_ERR_INTERNAL: return "internal error";
  }
  return "unknown status";
}

}  // extern "C"
