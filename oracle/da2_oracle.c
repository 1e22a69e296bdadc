/*
 * CPU oracle for the DraftAttention2 attention path.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, step-by-step restatement of what the method computes, written
 * from the paper: spatial blocks (Sec. 3.3 / App. C.2), average and max region
 * descriptors (Eq. "v2-descriptors"), the draft map (Def. 3.1, Eq. "v2-draft"),
 * ranking and precision tags (Algorithm 1), the operand quantisers (App. C.3)
 * and the phased mixed-precision attention with one shared online-softmax state
 * (Sec. 3.3 "Phased execution" / "Cross-precision accumulation", App. B.3, C.4).
 *
 * It shares no code with the CUDA library and must never be linked or called by
 * it.  Only tests, the smoke check and the CPU-baseline leg of the benchmark use
 * it.  Floating point is fp64 except where the paper fixes an fp32 quantity
 * (quantisation scales, codes, the fp32 softmax weights that get quantised):
 * there every operation is a single IEEE fp32 operation, in the order written.
 *
 * Layout conventions
 *   x        bf16 bits, [BH, N, d], raster token order u = (t*Hg + y)*Wg + x
 *   block a  = (t*nty + ty)*ntx + tx ; slot j = ly*tw + lx ; S = th*tw slots
 *   slot_token[a*S + j] = token index or -1 (padding of a ragged edge tile)
 *   "block order" arrays are [BH, R, S, d]; padding slots hold code 0.
 *
 * Parity pins live in tests/ (oracle vs. closed forms, brute force and bounds);
 * none of the functions below is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef int64_t i64;

/* ------------------------------------------------------------------ bf16 */
static float bf16_bits_to_f32(uint16_t b) {
  uint32_t u = (uint32_t)b << 16;
  float f;
  memcpy(&f, &u, 4);
  return f;
}

/* round-to-nearest-even fp32 -> bf16, returned as the fp32 value it denotes */
static float round_to_bf16(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  if ((u & 0x7fffffffu) > 0x7f800000u) return f; /* NaN */
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7fffu + lsb;
  u &= 0xffff0000u;
  memcpy(&f, &u, 4);
  return f;
}

/* ------------------------------------------------- small float formats */
/* OCP E4M3 (finite-only variant): 1 sign, 4 exponent (bias 7), 3 mantissa bits.
 * code 0x7f / 0xff are NaN; largest finite magnitude 448 (code 0x7e). */
static double e4m3_magnitude(int code7) { /* code7 in [0,126] */
  int e = code7 >> 3, m = code7 & 7;
  if (e == 0) return ldexp((double)m, -9);        /* subnormal: m * 2^-9 */
  return ldexp(1.0 + (double)m / 8.0, e - 7);
}

/* E2M1: 1 sign, 2 exponent, 1 mantissa: magnitudes 0,.5,1,1.5,2,3,4,6 */
static const double E2M1_MAG[8] = {0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0};

/* nearest entry of an ascending table; exact midpoints go to the even index;
 * anything beyond the last entry saturates to it. */
static int nearest_even_index(double mag, int n, double (*value)(int)) {
  int lo = 0, hi = n - 1;
  if (mag >= value(hi)) return hi;
  /* invariant: value(lo) <= mag < value(hi) */
  while (hi - lo > 1) {
    int mid = (lo + hi) / 2;
    if (mag >= value(mid)) lo = mid; else hi = mid;
  }
  double mid = 0.5 * (value(lo) + value(hi)); /* exact in fp64 */
  if (mag < mid) return lo;
  if (mag > mid) return hi;
  return (lo & 1) ? hi : lo;
}
static double e4m3_value_at(int i) { return e4m3_magnitude(i); }
static double e2m1_value_at(int i) { return E2M1_MAG[i]; }

/* cast_E4M3: round to nearest, ties to even code, saturate to +-448 */
uint8_t orc_cast_e4m3(float x) {
  if (isnan(x)) return 0x7f;
  int sign = signbit(x) ? 0x80 : 0;
  double mag = fabs((double)x);
  return (uint8_t)(sign | nearest_even_index(mag, 127, e4m3_value_at));
}
float orc_decode_e4m3(uint8_t c) {
  if ((c & 0x7f) == 0x7f) return NAN;
  double v = e4m3_magnitude(c & 0x7f);
  return (float)((c & 0x80) ? -v : v);
}
/* cast_E2M1: round to nearest, ties to even code, saturate to +-6 */
uint8_t orc_cast_e2m1(float x) {
  int sign = signbit(x) ? 0x8 : 0;
  double mag = isnan(x) ? 6.0 : fabs((double)x);
  return (uint8_t)(sign | nearest_even_index(mag, 8, e2m1_value_at));
}
float orc_decode_e2m1(uint8_t c) {
  double v = E2M1_MAG[c & 7];
  return (float)((c & 8) ? -v : v);
}

/* ------------------------------------------------------------------ plan */
/* Fixed th x tw spatial tiles inside each frame, ragged edge tiles padded.
 * Returns R = T * ceil(Hg/th) * ceil(Wg/tw).  slot_token: [R*th*tw], n_valid: [R].
 * Either output may be NULL (then only R is returned). */
int orc_plan(int T, int Hg, int Wg, int th, int tw, int32_t *slot_token, int32_t *n_valid) {
  int nty = (Hg + th - 1) / th, ntx = (Wg + tw - 1) / tw;
  int R = T * nty * ntx, S = th * tw;
  for (int t = 0; t < T; ++t)
    for (int ty = 0; ty < nty; ++ty)
      for (int tx = 0; tx < ntx; ++tx) {
        int a = (t * nty + ty) * ntx + tx, cnt = 0;
        for (int ly = 0; ly < th; ++ly)
          for (int lx = 0; lx < tw; ++lx) {
            int y = ty * th + ly, x = tx * tw + lx, j = ly * tw + lx;
            int tok = (y < Hg && x < Wg) ? (t * Hg + y) * Wg + x : -1;
            if (slot_token) slot_token[(i64)a * S + j] = tok;
            cnt += tok >= 0;
          }
        if (n_valid) n_valid[a] = cnt;
      }
  return R;
}

/* ------------------------------------------------- balanced ragged partition (App. C.2)
 * Every H x W frame is cut into R_f = ceil(HW / C) connected regions of balanced size (sizes differ by at
 * most one, so padding is below one block per frame, Eq. "ragged-padding"), and among candidate partitions
 * the one with the smallest total perimeter is taken (Eq. "region-perimeter").  The paper names neither the
 * candidates nor the order of tokens inside a block; this reading fixes both:
 *   - a candidate is a band order: the frame is cut into r bands along one axis (heights as equal as
 *     possible, the taller ones first); bands are walked one after the other, band b column by column
 *     (left to right for even b, right to left for odd b), the columns alternately downwards and upwards,
 *     the first column of every band downwards; "transposed" candidates do the same with rows and columns
 *     exchanged.  Cutting that order into R_f consecutive runs, the first HW mod R_f of them one token
 *     longer, gives the regions; slot j of a block is the j-th token of its run.
 *   - a candidate is admissible if every region is 4-connected; the admissible candidate with the smallest
 *     total perimeter wins, ties going to bands along rows first and then to fewer bands.  r = H (rows as
 *     bands) is always admissible, so a winner exists. */
static void band_order(int H, int W, int r, int transposed, int32_t *order /* [H*W] cell = y*W+x */) {
  int L = transposed ? W : H, M = transposed ? H : W; /* bands cut the axis of length L, columns run along M */
  int hb = L / r, extra = L % r, pos = 0, l0 = 0;
  for (int b = 0; b < r; ++b) {
    int h = hb + (b < extra);
    for (int i = 0; i < M; ++i) {
      int m = (b % 2 == 0) ? i : M - 1 - i;
      for (int k = 0; k < h; ++k) {
        int l = l0 + ((i % 2 == 0) ? k : h - 1 - k);
        order[pos++] = transposed ? (m * W + l) : (l * W + m);
      }
    }
    l0 += h;
  }
}

static int regions_connected(int H, int W, int Rf, const int32_t *region /* [H*W] */, int32_t *stack, uint8_t *seen) {
  for (int i = 0; i < H * W; ++i) seen[i] = 0;
  int comps = 0;
  for (int c0 = 0; c0 < H * W; ++c0) {
    if (seen[c0]) continue;
    ++comps;
    int top = 0;
    stack[top++] = c0;
    seen[c0] = 1;
    while (top) {
      int c = stack[--top], y = c / W, x = c % W;
      const int ny[4] = {y - 1, y + 1, y, y}, nx[4] = {x, x, x - 1, x + 1};
      for (int e = 0; e < 4; ++e) {
        if (ny[e] < 0 || ny[e] >= H || nx[e] < 0 || nx[e] >= W) continue;
        int c2 = ny[e] * W + nx[e];
        if (!seen[c2] && region[c2] == region[c]) { seen[c2] = 1; stack[top++] = c2; }
      }
    }
  }
  return comps == Rf;
}

static i64 total_perimeter(int H, int W, const int32_t *region) {
  i64 per = 0;
  for (int y = 0; y < H; ++y)
    for (int x = 0; x < W; ++x) {
      int c = y * W + x;
      per += (y == 0) + (y == H - 1) + (x == 0) + (x == W - 1);
      if (y + 1 < H && region[c + W] != region[c]) per += 2;
      if (x + 1 < W && region[c + 1] != region[c]) per += 2;
    }
  return per;
}

/* Returns R = T * R_f.  slot_token: [R*C] (-1 = padding), n_valid: [R]; choice[0..2] = (transposed, bands,
 * total perimeter of one frame).  Outputs may be NULL. */
int orc_plan_balanced(int T, int Hg, int Wg, int C, int32_t *slot_token, int32_t *n_valid, i64 *choice) {
  int HW = Hg * Wg, Rf = (HW + C - 1) / C, n = HW / Rf, rem = HW % Rf;
  int32_t *order = (int32_t *)malloc(sizeof(int32_t) * (size_t)HW), *best = (int32_t *)malloc(sizeof(int32_t) * (size_t)HW);
  int32_t *region = (int32_t *)malloc(sizeof(int32_t) * (size_t)HW), *stack = (int32_t *)malloc(sizeof(int32_t) * (size_t)HW);
  uint8_t *seen = (uint8_t *)malloc((size_t)HW);
  i64 best_per = -1;
  int best_t = 0, best_r = 0;
  for (int tr = 0; tr < 2; ++tr)
    for (int r = 1; r <= (tr ? Wg : Hg); ++r) {
      band_order(Hg, Wg, r, tr, order);
      for (int a = 0, pos = 0; a < Rf; ++a)
        for (int j = 0; j < n + (a < rem); ++j) region[order[pos++]] = a;
      if (!regions_connected(Hg, Wg, Rf, region, stack, seen)) continue;
      i64 per = total_perimeter(Hg, Wg, region);
      if (best_per < 0 || per < best_per) {
        best_per = per; best_t = tr; best_r = r;
        for (int i = 0; i < HW; ++i) best[i] = order[i];
      }
    }
  if (choice) { choice[0] = best_t; choice[1] = best_r; choice[2] = best_per; }
  for (int t = 0; t < T; ++t)
    for (int a = 0, pos = 0; a < Rf; ++a) {
      int na = n + (a < rem);
      for (int j = 0; j < C; ++j)
        if (slot_token) slot_token[((i64)t * Rf + a) * C + j] = j < na ? t * HW + best[pos + j] : -1;
      if (n_valid) n_valid[t * Rf + a] = na;
      pos += na;
    }
  free(order); free(best); free(region); free(stack); free(seen);
  return T * Rf;
}

/* Integer quotas from fractions of M candidates: cumulative round-half-up, so the
 * three counts always sum to round(sum of fractions * M) (App. C.1: integer quotas
 * T_p with sum T; the rounding rule is this implementation's reading). */
void orc_quotas(double f16, double f8, double f4, i64 M, i64 out[3]) {
  i64 c16 = (i64)floor(f16 * (double)M + 0.5);
  i64 c8 = (i64)floor((f16 + f8) * (double)M + 0.5);
  i64 c4 = (i64)floor((f16 + f8 + f4) * (double)M + 0.5);
  if (c16 > M) c16 = M;
  if (c8 > M) c8 = M;
  if (c4 > M) c4 = M;
  out[0] = c16;
  out[1] = c8 - c16;
  out[2] = c4 - c8;
}

/* ------------------------------------------------------------------ pool */
/* Eq. "v2-descriptors": per region, the mean over its valid tokens and the
 * channel-wise maximum; padding excluded (App. C.1). avg,mx: fp32 [BH,R,d]. */
void orc_pool(const uint16_t *x, i64 BH, i64 N, int d, int R, int S, const int32_t *slot_token,
              float *avg, float *mx) {
#pragma omp parallel for collapse(2) schedule(static)
  for (i64 bh = 0; bh < BH; ++bh)
    for (int a = 0; a < R; ++a)
      for (int c = 0; c < d; ++c) {
        double sum = 0.0;
        float m = -INFINITY;
        int n = 0;
        for (int j = 0; j < S; ++j) {
          int tok = slot_token[(i64)a * S + j];
          if (tok < 0) continue;
          float val = bf16_bits_to_f32(x[(bh * N + tok) * d + c]);
          sum += (double)val;
          if (val > m) m = val;
          ++n;
        }
        avg[(bh * R + a) * d + c] = (float)(sum / (double)n);
        mx[(bh * R + a) * d + c] = m;
      }
}

/* ----------------------------------------------------------------- draft */
/* Def. 3.1, Eq. "v2-draft": A = (1-lambda) softmax_row(Qavg Kavg^T * scale)
 *                             + lambda softmax_row(Qmax Kmax^T * scale),
 * both softmaxes over all R key regions.  A: fp32 [BH,R,R]. */
void orc_draft(const float *qavg, const float *qmax, const float *kavg, const float *kmax, i64 BH,
               int R, int d, double lambda, double scale, float *A) {
#pragma omp parallel for collapse(2) schedule(static)
  for (i64 bh = 0; bh < BH; ++bh)
    for (int a = 0; a < R; ++a) {
      double *s1 = (double *)malloc(sizeof(double) * 2 * (size_t)R), *s2 = s1 + R;
      double m1 = -INFINITY, m2 = -INFINITY;
      for (int b = 0; b < R; ++b) {
        double d1 = 0.0, d2 = 0.0;
        for (int c = 0; c < d; ++c) {
          d1 += (double)qavg[(bh * R + a) * d + c] * (double)kavg[(bh * R + b) * d + c];
          d2 += (double)qmax[(bh * R + a) * d + c] * (double)kmax[(bh * R + b) * d + c];
        }
        s1[b] = scale * d1;
        s2[b] = scale * d2;
        if (s1[b] > m1) m1 = s1[b];
        if (s2[b] > m2) m2 = s2[b];
      }
      double z1 = 0.0, z2 = 0.0;
      for (int b = 0; b < R; ++b) {
        s1[b] = exp(s1[b] - m1);
        s2[b] = exp(s2[b] - m2);
        z1 += s1[b];
        z2 += s2[b];
      }
      for (int b = 0; b < R; ++b)
        A[(bh * R + a) * (i64)R + b] = (float)((1.0 - lambda) * (s1[b] / z1) + lambda * (s2[b] / z2));
      free(s1);
    }
}

/* ------------------------------------------------------------------ rank */
typedef struct { float score; i64 index; } scored_t;
static int by_score_desc_then_index(const void *pa, const void *pb) {
  const scored_t *a = (const scored_t *)pa, *b = (const scored_t *)pb;
  if (a->score > b->score) return -1;
  if (a->score < b->score) return 1;
  return (a->index > b->index) - (a->index < b->index);
}
/* Algorithm 1 on n scores: stable descending order (ties -> lower index), the first
 * t16 entries get tag 16, the next t8 tag 8, the next t4 tag 4, the rest 0. */
static void tag_by_rank(const float *score, i64 n, i64 t16, i64 t8, i64 t4, uint8_t *tag) {
  scored_t *order = (scored_t *)malloc(sizeof(scored_t) * (size_t)n);
  for (i64 i = 0; i < n; ++i) { order[i].score = score[i]; order[i].index = i; }
  qsort(order, (size_t)n, sizeof(scored_t), by_score_desc_then_index);
  for (i64 r = 0; r < n; ++r) {
    uint8_t p = 0;
    if (r < t16) p = 16; else if (r < t16 + t8) p = 8; else if (r < t16 + t8 + t4) p = 4;
    tag[order[r].index] = p;
  }
  free(order);
}
/* per query-block row (the benchmark configurations' budget scope) */
void orc_rank_row(const float *A, i64 BH, int R, i64 k16, i64 k8, i64 k4, uint8_t *tags) {
#pragma omp parallel for schedule(static)
  for (i64 row = 0; row < BH * R; ++row) tag_by_rank(A + row * R, R, k16, k8, k4, tags + row * R);
}
/* across all R*R pairs of a head (Algorithm 1 as printed) */
void orc_rank_head(const float *A, i64 BH, int R, i64 T16, i64 T8, i64 T4, uint8_t *tags) {
#pragma omp parallel for schedule(dynamic)
  for (i64 bh = 0; bh < BH; ++bh)
    tag_by_rank(A + bh * R * (i64)R, (i64)R * R, T16, T8, T4, tags + bh * R * (i64)R);
}
/* Tags -> per-row lists in execution order (Sec. 3.3: NVFP4 segment, INT8 segment,
 * 16-bit segment), ids ascending inside a segment.  ids: int32 [rows, stride],
 * counts: int32 [rows, 3] = (n4, n8, n16). */
void orc_lists(const uint8_t *tags, i64 rows, int R, int stride, int32_t *ids, int32_t *counts) {
#pragma omp parallel for schedule(static)
  for (i64 row = 0; row < rows; ++row) {
    int pos = 0;
    const uint8_t tier[3] = {4, 8, 16};
    for (int s = 0; s < 3; ++s) {
      int n = 0;
      for (int b = 0; b < R; ++b)
        if (tags[row * R + b] == tier[s]) { if (pos < stride) ids[row * stride + pos] = b; ++pos; ++n; }
      counts[row * 3 + s] = n;
    }
    for (int p = pos; p < stride; ++p) ids[row * stride + p] = -1;
  }
}

/* ------------------------------------------------------------- quantisers */
/* INT8 Q/K (App. C.3): one fp32 scale per block, delta = amax/127 + 1e-7,
 * code = round-half-away(x/delta).  codes: int8 [BH,R,S,d]; delta: [BH,R]. */
void orc_quant_int8(const uint16_t *x, i64 BH, i64 N, int d, int R, int S, const int32_t *slot_token,
                    int8_t *codes, float *delta) {
#pragma omp parallel for collapse(2) schedule(static)
  for (i64 bh = 0; bh < BH; ++bh)
    for (int a = 0; a < R; ++a) {
      float amax = 0.0f;
      for (int j = 0; j < S; ++j) {
        int tok = slot_token[(i64)a * S + j];
        if (tok < 0) continue;
        for (int c = 0; c < d; ++c) {
          float v = fabsf(bf16_bits_to_f32(x[(bh * N + tok) * d + c]));
          if (v > amax) amax = v;
        }
      }
      volatile float q = amax / 127.0f;
      volatile float dl = q + 1e-7f;
      delta[bh * R + a] = dl;
      for (int j = 0; j < S; ++j) {
        int tok = slot_token[(i64)a * S + j];
        for (int c = 0; c < d; ++c) {
          int8_t code = 0;
          if (tok >= 0) {
            volatile float r = bf16_bits_to_f32(x[(bh * N + tok) * d + c]) / dl;
            code = (int8_t)roundf(r);
          }
          codes[((bh * R + a) * S + j) * d + c] = code;
        }
      }
    }
}

/* E4M3 V for the 8-bit path (App. C.3): per (head, channel) scale
 * delta_c = max_v |V_vc| / 2.25 over the whole head; all-zero channel -> codes 0, scale 0. */
void orc_quant_v_e4m3(const uint16_t *v, i64 BH, i64 N, int d, int R, int S, const int32_t *slot_token,
                      uint8_t *codes, float *delta_c) {
#pragma omp parallel for schedule(static)
  for (i64 bh = 0; bh < BH; ++bh) {
    for (int c = 0; c < d; ++c) {
      float vmax = 0.0f;
      for (i64 u = 0; u < N; ++u) {
        float val = fabsf(bf16_bits_to_f32(v[(bh * N + u) * d + c]));
        if (val > vmax) vmax = val;
      }
      volatile float dl = vmax / 2.25f;
      delta_c[bh * d + c] = dl;
    }
    for (int a = 0; a < R; ++a)
      for (int j = 0; j < S; ++j) {
        int tok = slot_token[(i64)a * S + j];
        for (int c = 0; c < d; ++c) {
          uint8_t code = 0;
          float dl = delta_c[bh * d + c];
          if (tok >= 0 && dl > 0.0f) {
            volatile float r = bf16_bits_to_f32(v[(bh * N + tok) * d + c]) / dl;
            code = orc_cast_e4m3(r);
          }
          codes[((bh * R + a) * S + j) * d + c] = code;
        }
      }
  }
}

/* E4M3 values of the 8-bit path with a GIVEN per-(head, channel) scale delta_c (App. C.3 takes
 * delta_c = max_v |V_vc| / 2.25 from the tensor itself; a caller may instead carry the scale of an
 * earlier, similar tensor over, e.g. of the previous denoising step: the cast is the same, only the
 * scale's origin differs).  code = cast_E4M3(fl32(V / delta_c)); delta_c = 0 marks a skipped channel. */
void orc_quant_v_e4m3_given(const uint16_t *v, i64 BH, i64 N, int d, int R, int S, const int32_t *slot_token,
                            const float *delta_c, uint8_t *codes) {
#pragma omp parallel for schedule(static)
  for (i64 bh = 0; bh < BH; ++bh)
    for (int a = 0; a < R; ++a)
      for (int j = 0; j < S; ++j) {
        int tok = slot_token[(i64)a * S + j];
        for (int c = 0; c < d; ++c) {
          uint8_t code = 0;
          float dl = delta_c[bh * d + c];
          if (tok >= 0 && dl > 0.0f) {
            volatile float r = bf16_bits_to_f32(v[(bh * N + tok) * d + c]) / dl;
            code = orc_cast_e4m3(r);
          }
          codes[((bh * R + a) * S + j) * d + c] = code;
        }
      }
}

/* per-head max |x| over all valid tokens, and the derived NVFP4 per-tensor scale
 * g = amax / 2688 (so the largest group scale encodes as 448); g = 1 for a zero head. */
void orc_nvfp4_global_scale(const uint16_t *x, i64 BH, i64 N, int d, float *g) {
#pragma omp parallel for schedule(static)
  for (i64 bh = 0; bh < BH; ++bh) {
    float amax = 0.0f;
    for (i64 i = 0; i < N * d; ++i) {
      float v = fabsf(bf16_bits_to_f32(x[bh * N * d + i]));
      if (v > amax) amax = v;
    }
    volatile float gg = amax / 2688.0f;
    g[bh] = amax > 0.0f ? gg : 1.0f;
  }
}

/* one NVFP4 group (Eq. "v2-nvfp4-quantization"): vals[n] -> local E4M3 scale + E2M1 codes */
static void nvfp4_group(const float *vals, int n, float g, uint8_t *sf_code, uint8_t *codes) {
  float gmax = 0.0f;
  for (int i = 0; i < n; ++i) {
    float a = fabsf(vals[i]);
    if (a > gmax) gmax = a;
  }
  volatile float six_g = 6.0f * g;
  volatile float ratio = gmax / six_g;
  uint8_t sc = orc_cast_e4m3(ratio);
  float sigma = orc_decode_e4m3(sc);
  *sf_code = sc;
  if (sigma == 0.0f) { /* a group whose encoded scale is zero is encoded as zero */
    for (int i = 0; i < n; ++i) codes[i] = 0;
    return;
  }
  volatile float step = g * sigma;
  for (int i = 0; i < n; ++i) {
    volatile float r = vals[i] / step;
    codes[i] = orc_cast_e2m1(r);
  }
}

/* NVFP4 for Q and K: groups of 16 consecutive channels of one token.
 * codes: uint8 (one 4-bit code per byte) [BH,R,S,d]; sf: E4M3 codes [BH,R,S,d/16]. */
void orc_quant_nvfp4_qk(const uint16_t *x, i64 BH, i64 N, int d, int R, int S, const int32_t *slot_token,
                        const float *g, uint8_t *codes, uint8_t *sf) {
  int ng = d / 16;
#pragma omp parallel for collapse(2) schedule(static)
  for (i64 bh = 0; bh < BH; ++bh)
    for (int a = 0; a < R; ++a)
      for (int j = 0; j < S; ++j) {
        int tok = slot_token[(i64)a * S + j];
        for (int gi = 0; gi < ng; ++gi) {
          float vals[16];
          for (int i = 0; i < 16; ++i)
            vals[i] = tok >= 0 ? bf16_bits_to_f32(x[(bh * N + tok) * d + gi * 16 + i]) : 0.0f;
          nvfp4_group(vals, 16, g[bh], &sf[((bh * R + a) * S + j) * ng + gi],
                      &codes[((bh * R + a) * S + j) * d + gi * 16]);
        }
      }
}

/* NVFP4 for V: groups of 16 consecutive key slots (16*gi .. 16*gi+15) of one block, per channel.
 * codes: [BH,R,S,d]; sf: [BH,R,S/16,d]. Padding slots count as 0. */
void orc_quant_nvfp4_v(const uint16_t *v, i64 BH, i64 N, int d, int R, int S, const int32_t *slot_token,
                       const float *g, uint8_t *codes, uint8_t *sf) {
  int ng = S / 16;
#pragma omp parallel for collapse(2) schedule(static)
  for (i64 bh = 0; bh < BH; ++bh)
    for (int a = 0; a < R; ++a)
      for (int gi = 0; gi < ng; ++gi)
        for (int c = 0; c < d; ++c) {
          float vals[16];
          uint8_t cc[16];
          for (int i = 0; i < 16; ++i) {
            int tok = slot_token[(i64)a * S + gi * 16 + i];
            vals[i] = tok >= 0 ? bf16_bits_to_f32(v[(bh * N + tok) * d + c]) : 0.0f;
          }
          nvfp4_group(vals, 16, g[bh], &sf[((bh * R + a) * ng + gi) * d + c], cc);
          for (int i = 0; i < 16; ++i) codes[((bh * R + a) * S + gi * 16 + i) * d + c] = cc[i];
        }
}

/* -------------------------------------------------------------- attention */
typedef struct {
  const uint16_t *q, *k, *v;        /* bf16 raster [BH,N,d] */
  i64 BH, N;
  int d, R, S;
  const int32_t *slot_token;
  const int32_t *ids, *counts;      /* lists: [BH*R, stride], [BH*R, 3] */
  int stride;
  const int8_t *q8, *k8;            /* INT8 codes, block order */
  const float *dq8, *dk8;           /* [BH,R] */
  const uint8_t *v8;                /* E4M3 codes, block order */
  const float *dv8;                 /* [BH,d] */
  const uint8_t *q4, *k4, *v4;      /* E2M1 codes, block order */
  const uint8_t *sfq, *sfk, *sfv;   /* E4M3 scale codes */
  const float *gq, *gk, *gv;        /* [BH] */
  double scale;
  int encoded_units;                /* 1: carry the 8-bit phase in encoded units (Enter/Exit) */
} attn_args_t;

/* optional per-row diagnostics over key tokens (raster index), used by the bound tests */
typedef struct {
  double *shat;    /* [N] reconstructed logits, NaN where not retained */
  double *h_at;    /* [N] running row maximum when the key's block was processed */
  double *what;    /* [N] locally quantised numerator weight (relative to h_at) */
  double *vhat;    /* [N*d] reconstructed values */
  int32_t *tier;   /* [N] 0/4/8/16 */
  double *h_final; /* [1] */
  double *ell;     /* [1] */
} attn_debug_t;

#define ETA_P8 0.0022326917f   /* probability dequantisation scale of the 8-bit path (App. C.3) */
#define OFFSET_P8 8.807        /* base-2 exponent offset, about log2(448) */

/* One query row u of block a against the row's list.  out: d fp32 values (already bf16-rounded). */
static void attention_row(const attn_args_t *A, i64 bh, int a, int ju, float *out, attn_debug_t *dbg) {
  const int d = A->d, S = A->S, R = A->R;
  const i64 N = A->N;
  const int tok_u = A->slot_token[(i64)a * S + ju];
  const i64 row = bh * R + a;
  const int n4 = A->counts[row * 3 + 0], n8 = A->counts[row * 3 + 1], n16 = A->counts[row * 3 + 2];
  double *U = (double *)calloc((size_t)d, sizeof(double));     /* numerator, common units */
  double *Uenc = (double *)calloc((size_t)d, sizeof(double));  /* 8-bit phase, encoded units */
  double h = -INFINITY, ell = 0.0, ell_enc = 0.0;
  const double amp8 = exp2(OFFSET_P8);
  int in_enc = 0;
  double shat[256]; /* S <= 256 */
  float w32[256];

  for (int pos = 0; pos < n4 + n8 + n16; ++pos) {
    const int tier = pos < n4 ? 4 : (pos < n4 + n8 ? 8 : 16);
    const int b = A->ids[row * A->stride + pos];
    const i64 qb = (bh * R + a) * (i64)S + ju, kb0 = (bh * R + b) * (i64)S;

    /* phase boundary handling for the encoded-units variant (Eq. "precision-state-conversion") */
    if (A->encoded_units) {
      if (tier == 8 && !in_enc) { /* Enter */
        for (int c = 0; c < d; ++c) {
          double dl = A->dv8[bh * d + c];
          Uenc[c] = dl > 0.0 ? U[c] / ((double)ETA_P8 * dl) : 0.0;
        }
        ell_enc = ell / (double)ETA_P8;
        in_enc = 1;
      } else if (tier != 8 && in_enc) { /* Exit */
        for (int c = 0; c < d; ++c) {
          double dl = A->dv8[bh * d + c];
          if (dl > 0.0) U[c] = (double)ETA_P8 * dl * Uenc[c];
        }
        ell = (double)ETA_P8 * ell_enc;
        in_enc = 0;
      }
    }

    /* 1. logits of the block's valid keys from the reconstructed operands */
    double bmax = -INFINITY;
    for (int jv = 0; jv < S; ++jv) {
      int tok_v = A->slot_token[(i64)b * S + jv];
      if (tok_v < 0) { shat[jv] = -INFINITY; continue; }
      double s;
      if (tier == 16) {
        double acc = 0.0;
        for (int c = 0; c < d; ++c)
          acc += (double)bf16_bits_to_f32(A->q[(bh * N + tok_u) * d + c]) *
                 (double)bf16_bits_to_f32(A->k[(bh * N + tok_v) * d + c]);
        s = A->scale * acc;
      } else if (tier == 8) {
        i64 acc = 0;
        for (int c = 0; c < d; ++c) acc += (i64)A->q8[qb * d + c] * (i64)A->k8[(kb0 + jv) * d + c];
        s = (double)A->dq8[bh * R + a] * (double)A->dk8[bh * R + b] * A->scale * (double)acc;
      } else {
        double acc = 0.0;
        for (int gi = 0; gi < d / 16; ++gi) {
          double part = 0.0;
          for (int i = 0; i < 16; ++i)
            part += (double)orc_decode_e2m1(A->q4[qb * d + gi * 16 + i]) *
                    (double)orc_decode_e2m1(A->k4[(kb0 + jv) * d + gi * 16 + i]);
          acc += (double)orc_decode_e4m3(A->sfq[qb * (d / 16) + gi]) *
                 (double)orc_decode_e4m3(A->sfk[(kb0 + jv) * (d / 16) + gi]) * part;
        }
        s = (double)A->gq[bh] * (double)A->gk[bh] * A->scale * acc;
      }
      shat[jv] = s;
      if (s > bmax) bmax = s;
    }
    if (bmax == -INFINITY) continue; /* cannot happen: every tile has a valid token */

    /* 2. running maximum first, then rescale the state */
    double hn = h > bmax ? h : bmax;
    double corr = (h == -INFINITY) ? 0.0 : exp(h - hn);
    for (int c = 0; c < d; ++c) { U[c] *= corr; Uenc[c] *= corr; }
    ell *= corr;
    ell_enc *= corr;
    h = hn;

    /* 3. fp32 weights; the denominator takes them before any conversion */
    for (int jv = 0; jv < S; ++jv) {
      if (shat[jv] == -INFINITY) { w32[jv] = 0.0f; continue; }
      w32[jv] = (float)exp(shat[jv] - h);
      if (in_enc) ell_enc += (double)w32[jv] * amp8; else ell += (double)w32[jv];
    }

    /* 4. numerator with the tier's operand formats */
    if (tier == 16) {
      for (int jv = 0; jv < S; ++jv) {
        int tok_v = A->slot_token[(i64)b * S + jv];
        if (tok_v < 0) continue;
        double wq = (double)round_to_bf16(w32[jv]);
        for (int c = 0; c < d; ++c) U[c] += wq * (double)bf16_bits_to_f32(A->v[(bh * N + tok_v) * d + c]);
        if (dbg) { dbg->what[tok_v] = wq; }
      }
    } else if (tier == 8) {
      for (int jv = 0; jv < S; ++jv) {
        int tok_v = A->slot_token[(i64)b * S + jv];
        if (tok_v < 0) continue;
        float amplified = (float)((double)w32[jv] * amp8);
        double pq = (double)orc_decode_e4m3(orc_cast_e4m3(amplified));
        for (int c = 0; c < d; ++c) {
          double dl = A->dv8[bh * d + c];
          double vq = (double)orc_decode_e4m3(A->v8[(kb0 + jv) * d + c]);
          if (in_enc) { if (dl > 0.0) Uenc[c] += pq * vq; }
          else U[c] += (double)ETA_P8 * pq * dl * vq;
        }
        if (dbg) dbg->what[tok_v] = (double)ETA_P8 * pq;
      }
    } else {
      for (int gi = 0; gi < S / 16; ++gi) {
        float gm = 0.0f;
        for (int i = 0; i < 16; ++i) if (w32[gi * 16 + i] > gm) gm = w32[gi * 16 + i];
        volatile float sp_in = 448.0f * gm;
        float sigma_p = orc_decode_e4m3(orc_cast_e4m3(sp_in));
        if (sigma_p == 0.0f) continue; /* zero-scale groups produce zeros */
        double pq[16];
        for (int i = 0; i < 16; ++i) {
          float r = (float)(2688.0 * (double)w32[gi * 16 + i] / (double)sigma_p);
          pq[i] = (double)orc_decode_e2m1(orc_cast_e2m1(r));
          int tok_v = A->slot_token[(i64)b * S + gi * 16 + i];
          if (dbg && tok_v >= 0) dbg->what[tok_v] = (double)sigma_p / 2688.0 * pq[i];
        }
        for (int c = 0; c < d; ++c) {
          double part = 0.0;
          for (int i = 0; i < 16; ++i)
            part += pq[i] * (double)orc_decode_e2m1(A->v4[(kb0 + gi * 16 + i) * d + c]);
          double sv = (double)orc_decode_e4m3(A->sfv[((bh * R + b) * (S / 16) + gi) * d + c]);
          U[c] += (double)A->gv[bh] / 2688.0 * (double)sigma_p * sv * part;
        }
      }
    }

    if (dbg)
      for (int jv = 0; jv < S; ++jv) {
        int tok_v = A->slot_token[(i64)b * S + jv];
        if (tok_v < 0) continue;
        dbg->shat[tok_v] = shat[jv];
        dbg->h_at[tok_v] = h;
        dbg->tier[tok_v] = tier;
        for (int c = 0; c < d; ++c) {
          double vh;
          if (tier == 16) vh = (double)bf16_bits_to_f32(A->v[(bh * N + tok_v) * d + c]);
          else if (tier == 8) vh = (double)A->dv8[bh * d + c] * (double)orc_decode_e4m3(A->v8[(kb0 + jv) * d + c]);
          else vh = (double)A->gv[bh] * (double)orc_decode_e4m3(A->sfv[((bh * R + b) * (S / 16) + jv / 16) * d + c]) *
                    (double)orc_decode_e2m1(A->v4[(kb0 + jv) * d + c]);
          dbg->vhat[(i64)tok_v * d + c] = vh;
        }
      }
  }
  if (in_enc) { /* Exit after the last block if the 8-bit phase was the final one */
    for (int c = 0; c < d; ++c) {
      double dl = A->dv8[bh * d + c];
      if (dl > 0.0) U[c] = (double)ETA_P8 * dl * Uenc[c];
    }
    ell = (double)ETA_P8 * ell_enc;
  }
  /* 5. one normalisation; a row without retained keys returns zero (App. C.1) */
  for (int c = 0; c < d; ++c) out[c] = ell > 0.0 ? round_to_bf16((float)(U[c] / ell)) : 0.0f;
  if (dbg) { *dbg->h_final = h; *dbg->ell = ell; }
  free(U);
  free(Uenc);
}

/* Phased mixed-precision attention for nsel selected query blocks.
 * sel: [nsel,2] = (flat head index, query block).  out: fp32 [nsel,S,d]; padding query slots 0. */
void orc_attention(const uint16_t *q, const uint16_t *k, const uint16_t *v, i64 BH, i64 N, int d, int R, int S,
                   const int32_t *slot_token, const int32_t *ids, const int32_t *counts, int stride,
                   const int8_t *q8, const int8_t *k8, const float *dq8, const float *dk8,
                   const uint8_t *v8, const float *dv8,
                   const uint8_t *q4, const uint8_t *k4, const uint8_t *v4,
                   const uint8_t *sfq, const uint8_t *sfk, const uint8_t *sfv,
                   const float *gq, const float *gk, const float *gv,
                   double scale, int encoded_units, const int32_t *sel, int nsel, float *out) {
  attn_args_t A = {q, k, v, BH, N, d, R, S, slot_token, ids, counts, stride, q8, k8, dq8, dk8, v8, dv8,
                   q4, k4, v4, sfq, sfk, sfv, gq, gk, gv, scale, encoded_units};
#pragma omp parallel for collapse(2) schedule(dynamic)
  for (int i = 0; i < nsel; ++i)
    for (int ju = 0; ju < S; ++ju) {
      float *o = out + ((i64)i * S + ju) * d;
      if (slot_token[(i64)sel[2 * i + 1] * S + ju] < 0) { for (int c = 0; c < d; ++c) o[c] = 0.0f; continue; }
      attention_row(&A, sel[2 * i], sel[2 * i + 1], ju, o, NULL);
    }
}

/* Same, one query row, with diagnostics over key tokens (arrays sized N, N, N, N*d, N, 1, 1). */
void orc_attention_row_debug(const uint16_t *q, const uint16_t *k, const uint16_t *v, i64 BH, i64 N, int d, int R,
                             int S, const int32_t *slot_token, const int32_t *ids, const int32_t *counts,
                             int stride, const int8_t *q8, const int8_t *k8, const float *dq8, const float *dk8,
                             const uint8_t *v8, const float *dv8, const uint8_t *q4, const uint8_t *k4,
                             const uint8_t *v4, const uint8_t *sfq, const uint8_t *sfk, const uint8_t *sfv,
                             const float *gq, const float *gk, const float *gv, double scale, i64 bh, int a,
                             int ju, float *out, double *shat, double *h_at, double *what, double *vhat,
                             int32_t *tier, double *h_final, double *ell) {
  attn_args_t A = {q, k, v, BH, N, d, R, S, slot_token, ids, counts, stride, q8, k8, dq8, dk8, v8, dv8,
                   q4, k4, v4, sfq, sfk, sfv, gq, gk, gv, scale, 0};
  attn_debug_t D = {shat, h_at, what, vhat, tier, h_final, ell};
  for (i64 i = 0; i < N; ++i) { shat[i] = NAN; h_at[i] = NAN; what[i] = 0.0; tier[i] = 0; }
  attention_row(&A, bh, a, ju, out, &D);
}

/* Dense softmax attention in fp64 on the stored bf16 inputs (Eq. "v2-dense"),
 * for the query tokens of selected blocks.  out: fp64 [nsel,S,d]; padding slots 0. */
void orc_dense(const uint16_t *q, const uint16_t *k, const uint16_t *v, i64 BH, i64 N, int d, int S,
               const int32_t *slot_token, double scale, const int32_t *sel, int nsel, double *out) {
  (void)BH;
#pragma omp parallel for collapse(2) schedule(dynamic)
  for (int i = 0; i < nsel; ++i)
    for (int ju = 0; ju < S; ++ju) {
      i64 bh = sel[2 * i];
      int tok_u = slot_token[(i64)sel[2 * i + 1] * S + ju];
      double *o = out + ((i64)i * S + ju) * d;
      for (int c = 0; c < d; ++c) o[c] = 0.0;
      if (tok_u < 0) continue;
      double *s = (double *)malloc(sizeof(double) * (size_t)N);
      double m = -INFINITY, z = 0.0;
      for (i64 u = 0; u < N; ++u) {
        double acc = 0.0;
        for (int c = 0; c < d; ++c)
          acc += (double)bf16_bits_to_f32(q[(bh * N + tok_u) * d + c]) *
                 (double)bf16_bits_to_f32(k[(bh * N + u) * d + c]);
        s[u] = scale * acc;
        if (s[u] > m) m = s[u];
      }
      for (i64 u = 0; u < N; ++u) { s[u] = exp(s[u] - m); z += s[u]; }
      for (i64 u = 0; u < N; ++u) {
        double p = s[u] / z;
        for (int c = 0; c < d; ++c) o[c] += p * (double)bf16_bits_to_f32(v[(bh * N + u) * d + c]);
      }
      free(s);
    }
}
