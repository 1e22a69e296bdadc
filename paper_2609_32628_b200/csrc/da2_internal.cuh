// Internal declarations shared by the da2 kernels (host plan, device parameter block, small helpers).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "da2.h"

namespace da2 {

constexpr int kSlots = 64;      // tokens per block: one 8 x 8 spatial tile of one frame
constexpr int kTile = 8;
constexpr int kSfAtomBytes = 512;  // one scale-factor atom: 128 rows x 4 groups of E4M3 codes

// device status word values (workspace off_status[0])
constexpr int kDevOk = 0;
constexpr int kDevTimeout = 1;
constexpr int kDevBadList = 2;

// Plain-old-data parameter block handed to every kernel by value.
struct Params {
  int B, H, T, Hg, Wg, d;
  int nty, ntx, R_f, R;
  long long N;              // video tokens per head
  int P, Rp, Rt;            // prefix tokens, prefix blocks (ceil(P / 64)), blocks per head R + Rp
  long long Ntot;           // tokens per head in the tensors: P prefix tokens, then the N video tokens
  int row_stride;           // id entries reserved per video row (ROW scope)
  // balanced ragged partition (App. C.2): 0 = fixed 8 x 8 tiles; else the chosen band order and the run lengths
  int part, part_tr, part_bands, part_n, part_rem;
  int BH;
  int rank_scope;
  int tier_active[3];       // 0: NVFP4, 1: INT8/E4M3, 2: BF16
  long long quota[3];       // k4, k8, k16
  long long ids_per_head;
  float lambda, scale;
  uint32_t qrec_bytes[3], kvrec_bytes[3];
  // resolved device pointers into the workspace
  int *status;
  uint32_t *amax;           // [BH][4]
  uint32_t *vmax;           // [BH][d]
  float *gscale;            // [BH][4]
  float *desc[4];           // Qavg, Qmax, Kavg, Kmax [BH][R][d]
  float *logits[2];         // [BH][R][R]
  float *map;               // [BH][R][R]
  int *counts;              // [BH][R][4]
  uint16_t *ids;            // [BH][ids_per_head]
  uint32_t *select;         // HEAD-scope scratch
  uint8_t *qrec[3], *kvrec[3];
  float *dq8, *dk8, *dv8;
  uint16_t *order;          // [BH][2*ceil(R/2)] query blocks by decreasing list length
  // region table of one frame, written with the operand records: cell (y * Wg + x) of slot j of region r, and the
  // region's slot-valid mask; the attention kernel looks tokens up here instead of carrying the region arithmetic
  int *region_cell;               // [R_f][64]
  unsigned long long *region_mask;  // [R_f]
};

// number of valid rows / columns of tile (ty, tx) and the 64-bit slot-valid mask of block a
// (blocks R .. R + Rp - 1 are runs of 64 consecutive prefix tokens; the last one may be short)
__host__ __device__ inline unsigned long long block_valid_mask(const Params &p, int a) {
  if (a >= p.R) {
    const int rem = p.P - (a - p.R) * kSlots;
    return rem >= kSlots ? ~0ull : ((1ull << rem) - 1ull);
  }
  int r = a % p.R_f;
  if (p.part) {  // a run of the band order: its n or n + 1 tokens fill the first slots
    const int na = p.part_n + (r < p.part_rem);
    return na >= kSlots ? ~0ull : ((1ull << na) - 1ull);
  }
  int ty = r / p.ntx, tx = r % p.ntx;
  int vr = min(kTile, p.Hg - ty * kTile), vc = min(kTile, p.Wg - tx * kTile);
  unsigned long long rowbits = (vc >= 8) ? 0xffull : ((1ull << vc) - 1ull);
  unsigned long long m = 0;
  for (int ly = 0; ly < vr; ++ly) m |= rowbits << (8 * ly);
  return m;
}

// token index (row of a head's [P + N, d] tensor) of slot j of block a: prefix tokens come first, then the video
// tokens in raster order (caller checks validity with the mask)
__host__ __device__ inline long long slot_token(const Params &p, int a, int j) {
  if (a >= p.R) return (long long)(a - p.R) * kSlots + j;
  int t = a / p.R_f, r = a % p.R_f;
  if (p.part) {
    // Band order: the frame is cut into part_bands bands along one axis (the taller ones first); band b is walked
    // column by column (forwards for even b, backwards for odd b), the columns alternately down and up; region r is
    // the r-th run of that order, slot j its j-th cell.
    const int L = p.part_tr ? p.Wg : p.Hg, M = p.part_tr ? p.Hg : p.Wg;
    const int hb = L / p.part_bands, extra = L % p.part_bands;
    int pos = r * p.part_n + min(r, p.part_rem) + j;
    const int big = extra * (hb + 1) * M;
    int b, h, q;
    if (pos < big) { h = hb + 1; b = pos / (h * M); q = pos - b * h * M; }
    else { h = hb; pos -= big; b = pos / (h * M); q = pos - b * h * M; b += extra; }
    const int l0 = b * hb + min(b, extra);
    const int i = q / h, k = q - i * h;
    const int m = (b & 1) ? M - 1 - i : i;
    const int l = l0 + ((i & 1) ? h - 1 - k : k);
    const int cell = p.part_tr ? m * p.Wg + l : l * p.Wg + m;
    return p.P + (long long)t * p.Hg * p.Wg + cell;
  }
  int ty = r / p.ntx, tx = r % p.ntx;
  int y = ty * kTile + (j >> 3), x = tx * kTile + (j & 7);
  return p.P + ((long long)t * p.Hg + y) * p.Wg + x;
}

// operand records per head and tier: the 16-bit tier also holds the prefix blocks
__host__ __device__ inline int rec_blocks(const Params &p, int tier) { return tier == 2 ? p.Rt : p.R; }

// kernel launchers (each returns the cudaError_t of its launch)
cudaError_t launch_pool(const Params &p, const __nv_bfloat16 *q, const __nv_bfloat16 *k, const __nv_bfloat16 *v,
                        cudaStream_t st, int *launches);
cudaError_t launch_draft(const Params &p, cudaStream_t st, int *launches);
cudaError_t launch_rank(const Params &p, cudaStream_t st, int *launches);
cudaError_t launch_map_rows(const Params &p, cudaStream_t st, int *launches);
cudaError_t launch_order(const Params &p, cudaStream_t st, int *launches);
cudaError_t launch_prefix_rows(const Params &p, cudaStream_t st, int *launches);
cudaError_t launch_prep(const Params &p, const __nv_bfloat16 *q, const __nv_bfloat16 *k, const __nv_bfloat16 *v,
                        cudaStream_t st, int *launches, bool pool = false);
cudaError_t launch_attention(const Params &p, __nv_bfloat16 *out, cudaStream_t st, int *launches);
cudaError_t launch_bounded_wait_probe(int *status, long long limit_cycles, cudaStream_t st);
cudaError_t launch_quantiser_selfcheck(int mode, int n_divisors, uint32_t seed, unsigned long long *out, cudaStream_t st);

}  // namespace da2

struct da2_plan {
  da2_config_t cfg;
  da2_plan_info_t info;
  float *g_host[3];       // optional caller-provided NVFP4 per-tensor scales (copied), or nullptr
  uint64_t off_region_cell, off_region_mask;  // workspace offsets of the region table (internal)
};
