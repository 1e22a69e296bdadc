/*
 * da2 -- DraftAttention2 attention hot path for NVIDIA B200 (sm_100a), C ABI.
 *
 * Low-resolution-guided block selection with mixed-precision block-sparse attention:
 *   da2_plan          host only: spatial tiling, quotas, workspace layout      (Sec. 3.3, App. C.1/C.2)
 *   da2_prepare       device: pool -> draft map -> rank/tag/lists -> operand quantisation
 *                                                                    (Eq. v2-descriptors, Def. 3.1, Alg. 1, App. C.3)
 *   da2_attention_fwd device: one phased kernel, NVFP4 -> INT8/E4M3 -> BF16 segments sharing one
 *                     online-softmax state and one output accumulator          (Sec. 3.3, App. C.4)
 *
 * Conventions
 *   - q, k, v, out: DEVICE pointers, contiguous bf16 [B, H, P + N, head_dim]: first the P = n_prefix prefix (text)
 *     tokens, if any, then the N = T*Hg*Wg video tokens in raster order u = (t*Hg + y)*Wg + x; 16-byte aligned.
 *     out must not alias the inputs.
 *   - workspace: DEVICE pointer, 256-byte aligned, at least da2_plan_info().workspace_bytes long.  The caller owns
 *     all device memory; the library allocates none and keeps no device state between calls (one exception:
 *     da2_draft_map_noalloc, which owns a fixed scratch array, see there).
 *   - stream: a cudaStream_t passed as void* (NULL = default stream).  da2_prepare and da2_attention_fwd only
 *     enqueue work and never synchronise.
 *   - Errors are return codes.  Argument errors are detected before any launch.  A device-side bounded wait that
 *     gives up records a code in the workspace status word; da2_device_status reports it.
 *   - The plan is host memory owned by the library until da2_plan_destroy; it is immutable (no call writes to it,
 *     so threads may share one) and may be reused for any number of calls with the same shapes and budgets (the
 *     partition is reused across layers and steps).
 *   - Limits: B*H <= 32767 and R = T*ceil(Hg/8)*ceil(Wg/8) <= 16384; beyond them da2_plan returns
 *     DA2_ERR_UNSUPPORTED.
 */
#ifndef DA2_H_
#define DA2_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  DA2_OK = 0,
  DA2_ERR_INVALID_ARG = 1,
  DA2_ERR_UNSUPPORTED = 2,
  DA2_ERR_WORKSPACE_TOO_SMALL = 3,
  DA2_ERR_CUDA = 4,
  DA2_ERR_TIMEOUT = 5,
  DA2_ERR_INTERNAL = 6
} da2_status_t;

/* Scope of the shared ranking (Alg. 1).  ROW: every query-block row keeps the same number of key blocks per
 * precision (the benchmark configurations).  HEAD: one ranking over all R*R region pairs of a head, as printed in
 * Alg. 1, so rows may keep different numbers of blocks, possibly none. */
typedef enum { DA2_RANK_ROW = 0, DA2_RANK_HEAD = 1 } da2_rank_scope_t;

/* How a latent frame is cut into regions (one region = one block of 64 slots).
 * TILES: fixed 8 x 8 spatial tiles, ragged edge tiles padded (the benchmark configurations).
 * BALANCED: the ragged partition of App. C.2: R_f = ceil(Hg*Wg / capacity) connected regions per frame whose token
 * counts differ by at most one (less than one block of padding per frame, Eq. "ragged-padding"), chosen with the
 * smallest total perimeter (Eq. "region-perimeter") among band-order candidates: the frame is cut into bands along
 * one axis, the bands are walked column by column in alternating directions, and that order is cut into R_f runs;
 * slot j of a block is the j-th token of its run. */
typedef enum { DA2_PARTITION_TILES = 0, DA2_PARTITION_BALANCED = 1 } da2_partition_t;

typedef struct {
  int32_t B, H, T, Hg, Wg, head_dim; /* head_dim in {64, 128} */
  int32_t tile_h, tile_w;            /* spatial tile of one block; only 8 x 8 is supported */
  double frac16, frac8, frac4;       /* budgets as fractions of key blocks: bf16 / INT8+E4M3 / NVFP4; sum <= 1 */
  float lambda;                      /* weight of the max-pooled draft branch in [0,1] (Def. 3.1) */
  float softmax_scale;               /* <= 0 selects 1/sqrt(head_dim) */
  int32_t rank_scope;                /* da2_rank_scope_t */
  int32_t n_prefix;                  /* P >= 0 prefix (text) tokens in front of the video tokens (App. C.1: prefix
                                        interactions lie outside the region budget).  Every video query keeps all
                                        prefix keys and every prefix query attends to all keys, both in the 16-bit
                                        tier; prefix tokens form ceil(P/64) blocks numbered after the video regions.
                                        Needs rank_scope = DA2_RANK_ROW.  0 = no prefix */
  const float *g_q, *g_k, *g_v;      /* optional HOST arrays [B*H]: NVFP4 per-tensor scales (App. C.3, g_X); NULL =
                                        derived per head as amax/2688.  Copied into the plan. */
  int32_t partition;                 /* da2_partition_t */
  int32_t capacity;                  /* block capacity C of the balanced partition; only 64 is supported (ignored
                                        for DA2_PARTITION_TILES) */
} da2_config_t;

typedef struct da2_plan da2_plan_t;

/* Everything a caller (or a parity harness) needs to size and read the workspace.  Offsets are bytes from the
 * workspace base.  "tier" index: 0 = NVFP4 (4-bit), 1 = INT8/E4M3 (8-bit), 2 = BF16 (16-bit). */
typedef struct {
  int32_t B, H, T, Hg, Wg, head_dim, tile_h, tile_w;
  int32_t nty, ntx, R_f, R, S;       /* tiles per frame, blocks per head, slots per block (64) */
  int64_t N;
  int32_t rank_scope;
  int32_t tier_active[3];            /* 1 if the tier has a non-zero quota */
  int64_t quota[3];                  /* (k4, k8, k16): per row (ROW scope) or per head (HEAD scope) */
  int64_t ids_per_head;              /* uint16 entries of the id array belonging to one head */
  float lambda, softmax_scale;
  uint64_t workspace_bytes;
  uint64_t off_status;               /* int32[64]: [0] status code, [1..] diagnostics */
  uint64_t off_amax;                 /* uint32[BH][4]: fp32 bit patterns of max|Q|, max|K|, max|V| per head */
  uint64_t off_vmax;                 /* uint32[BH][d]: fp32 bit patterns of max_v |V_vc| */
  uint64_t off_gscale;               /* fp32[BH][4]: NVFP4 per-tensor scales g_Q, g_K, g_V */
  uint64_t off_desc[4];              /* fp32[BH][R][d]: Qavg, Qmax, Kavg, Kmax */
  uint64_t off_logits[2];            /* fp32[BH][R][R]: draft logits of the average / max branch (scratch) */
  uint64_t off_map;                  /* fp32[BH][R][R]: draft map A (Def. 3.1) */
  uint64_t off_counts;               /* int32[BH][R][4]: (n4, n8, n16, offset of the row's ids inside its head) */
  uint64_t off_ids;                  /* uint16[BH][ids_per_head]: key-block ids, per row 4-bit | 8-bit | 16-bit
                                        segments, ascending inside a segment */
  uint64_t off_select;               /* scratch of the HEAD-scope selection */
  uint64_t off_qrec[3];              /* per tier: Q operand records [BH][R][qrec_bytes] */
  uint64_t off_kvrec[3];             /* per tier: K + V operand records [BH][R][kvrec_bytes] */
  uint32_t qrec_bytes[3], kvrec_bytes[3];
  uint64_t off_dq8, off_dk8;         /* fp32[BH][R]: INT8 block scales of Q and K */
  uint64_t off_dv8;                  /* fp32[BH][d]: E4M3 per-channel scale of V */
  int32_t n_prefix, R_prefix;        /* prefix tokens and their blocks, ceil(n_prefix / 64); with a prefix, rows and
                                        blocks R .. R + R_prefix - 1 are the prefix's: counts is int32[BH][R +
                                        R_prefix][4], the 16-bit records cover R + R_prefix blocks per head, and
                                        tier_active[2] is set */
  int32_t partition;                 /* da2_partition_t; for the balanced partition R_f = ceil(Hg*Wg/64) and: */
  int32_t part_transposed, part_bands; /* the chosen band order: bands along columns (1) or rows (0), their number */
  int32_t part_n, part_rem;          /* region r of a frame holds part_n + (r < part_rem) tokens, in its first slots */
  int64_t part_perimeter;            /* total perimeter of one frame's regions */
  int32_t row_stride;                /* ROW scope: id entries reserved per video row (its offset is row * row_stride) */
  uint64_t off_order;                /* uint16[BH][2*ceil(R/2)]: query blocks of a head by decreasing list length
                                        (ties: lower index first; 0xFFFF pads an odd R), written in HEAD scope only
                                        (per-row budgets: equal lengths, blocks 2p and 2p+1).  Scheduling only: the
                                        attention kernel gives CTA p of a head the blocks order[2p], order[2p+1],
                                        so that its two rows are equally long (the paper has no counterpart) */
} da2_plan_info_t;

/*
 * Operand record layouts (what da2_prepare writes and da2_attention_fwd streams into shared memory unchanged).
 * A "K-major image" of a [rows x kbytes] matrix stores 16-byte chunks: chunk (kc, r) at byte (kc*rows + r)*16,
 * i.e. 8 x 16 B core matrices, row-group stride 128 B, K-chunk stride rows*16 B.
 *   Q record, tier 2: image of bf16 [64 slots x d]                      (128*d/8 ... = 2*64*d bytes)
 *             tier 1: image of int8 [64 x d]                            (64*d bytes)
 *             tier 0: image of packed E2M1 [64 x d/2 bytes], then d/64 scale atoms of 512 B
 *   KV record: K part exactly like the Q record of the tier, then the V part:
 *             tier 2: image of bf16 V^T [d channels x 64 slots]
 *             tier 1: image of E4M3 V^T [d x 64]
 *             tier 0: image of packed E2M1 V^T [d x 32 bytes], then one 512 B scale atom
 *   Packed E2M1: element 2i in the low nibble of byte i.  Scale atom (E4M3 codes, one per 16 elements along the
 *   reduction dimension): byte (row%32)*16 + (row/32)*4 + group; Q/K atoms repeat rows 0..63 as rows 64..127.
 *   Padding slots of ragged edge tiles hold zeros.
 */

/* Builds the plan.  Host only; no CUDA call.  cfg and *plan_out must be non-NULL. */
da2_status_t da2_plan(const da2_config_t *cfg, da2_plan_t **plan_out);

/* Fills *info.  Host only. */
da2_status_t da2_plan_info(const da2_plan_t *plan, da2_plan_info_t *info);

/* The token-to-region map (Sec. 3.3: regions packed into contiguous blocks; the inverse map restores the output
 * order): index, within one head's [n_prefix + N] token sequence, of the token that slot `slot` (0..63) of block
 * `block` (0 .. R + R_prefix - 1) holds; -1 for a padding slot, -2 for arguments out of range.  Host only. */
int64_t da2_plan_slot_token(const da2_plan_t *plan, int32_t block, int32_t slot);

/* Pool, draft map, ranking, lists and operand records for (q, k, v) into workspace.  Enqueues on stream. */
da2_status_t da2_prepare(const da2_plan_t *plan, const void *q, const void *k, const void *v, void *workspace,
                         size_t workspace_bytes, void *stream);

/* Operands only.  The paper reuses the token-to-region partition across layers and denoising steps (Sec. 3.3,
 * "Fused quantization and reordering"): that is the plan object, which any number of calls may share.  This entry
 * point goes one step further on the caller's responsibility (the paper has no counterpart): it recomputes the
 * statistics, scales and operand records of (q, k, v) in a workspace that an earlier da2_prepare with the same plan
 * filled, and leaves that call's draft map, counts and id lists untouched, so that the selection of one call can
 * serve a later one.  Same argument rules as da2_prepare; the region descriptors are refreshed as a by-product.  In a
 * workspace that no da2_prepare has filled there are no lists: da2_attention_fwd then reads undefined ids (an id
 * out of range is reported through the status word, its row's output is undefined).  Enqueues on stream. */
da2_status_t da2_refresh_operands(const da2_plan_t *plan, const void *q, const void *k, const void *v,
                                  void *workspace, size_t workspace_bytes, void *stream);

/* Single-pass preparation under known quantiser statistics (Sec. 3.3, "Fused quantization and reordering": spatial
 * gathering, average- and max-pooling and quantisation fused so that the token features cross global memory once).
 * da2_prepare needs two passes over Q, K, V, because the NVFP4 per-tensor scales g_X and the E4M3 per-channel value
 * scales delta_c^V (App. C.3) are statistics of the whole head that must exist before any block is quantised.  This
 * call does not derive them: it quantises with the scales that are in the workspace -- left there by an earlier
 * da2_prepare / da2_refresh_operands with this plan, typically for the previous denoising step or layer, whose
 * activations have nearly the same range -- and writes region descriptors and every operand record in ONE pass
 * (INT8 block scales are local to a block and are always derived).  A value beyond the carried-over range saturates
 * in its format exactly as the casts define.  reselect != 0: the draft map, the ranking and the lists are then
 * recomputed from the new descriptors; reselect == 0: the earlier selection is kept (as da2_refresh_operands does).
 * The scales and statistics in the workspace are left untouched, so da2_attention_fwd dequantises with the scales
 * the records were made with.  Same argument rules as da2_prepare.  Enqueues on stream. */
da2_status_t da2_prepare_cached_scales(const da2_plan_t *plan, const void *q, const void *k, const void *v,
                                       void *workspace, size_t workspace_bytes, int32_t reselect, void *stream);

/* Phased mixed-precision block-sparse attention.  workspace must have been filled by da2_prepare for the same
 * q, k, v (ordering on the same stream is enough).  Rows whose list is empty give zeros (App. C.1). */
da2_status_t da2_attention_fwd(const da2_plan_t *plan, const void *q, const void *k, const void *v,
                               const void *workspace, void *out, void *stream);

/* The whole call on HOST tensors (the paper has no counterpart: packaging).  hq, hk, hv, hout: HOST pointers, bf16
 * [B, H, n_prefix + N, head_dim], ideally pinned (page-locked) so that the copies run asynchronously; arena: DEVICE
 * memory, 256-byte aligned, at least da2_attention_host_arena_bytes() long, owned by the caller (the library
 * allocates no device memory; it creates three streams and a few events for the duration of the call).  Heads are
 * independent, so the call is cut into groups of heads (n_groups > 0: that many nearly equal groups; 0: small groups at
 * both ends, large ones in between) whose host-to-device copies, kernels and device-to-host copies overlap on two
 * device slots.  Synchronous: returns after the last copy; the return value includes the device status of every
 * group (DA2_ERR_TIMEOUT / DA2_ERR_INTERNAL).  Caller-fixed g_q/g_k/g_v are not supported here
 * (DA2_ERR_UNSUPPORTED).  The result is bit-identical to da2_prepare + da2_attention_fwd on the whole tensors. */
da2_status_t da2_attention_host_arena_bytes(const da2_config_t *cfg, int32_t n_groups, size_t *bytes_out);
da2_status_t da2_attention_host(const da2_config_t *cfg, const void *hq, const void *hk, const void *hv, void *hout,
                                void *arena, size_t arena_bytes, int32_t n_groups);

/* Synchronises stream, reads the workspace status word; DA2_OK, DA2_ERR_TIMEOUT or DA2_ERR_INTERNAL. */
da2_status_t da2_device_status(const da2_plan_t *plan, const void *workspace, void *stream);

/* Number of kernels that the CALLING THREAD's last da2_prepare / da2_refresh_operands / da2_attention_fwd enqueued
 * (launch accounting; kept per thread, so the plan stays immutable).  plan must be non-NULL. */
int32_t da2_last_launch_count(const da2_plan_t *plan);

/* Failure-path probe (the paper has no counterpart; it exists so that the bounded device-side waits can be tested
 * without faulting or hanging a GPU).  Enqueues one small kernel that waits, through the same bounded wait the
 * attention kernel uses, on a barrier that nothing ever completes; after limit_cycles GPU clock cycles
 * (1 .. 2e9) the wait gives up, the kernel writes the time-out code into the workspace status word and returns
 * normally.  da2_device_status then reports DA2_ERR_TIMEOUT; the next da2_prepare clears the word. */
da2_status_t da2_probe_bounded_wait(const da2_plan_t *plan, void *workspace, int64_t limit_cycles, void *stream);

/* Arithmetic self-check of the operand quantisers (diagnostic; the paper has no counterpart).  The quantisers of
 * App. C.3 divide every element by a scale; the kernels obtain that quotient from a reciprocal taken once per scale and
 * two fused multiply-adds, and round INT8 codes half away from zero by one addition and a truncation.  This call
 * compares both, on the device and with the very device functions the kernels use, against the IEEE division and
 * against roundf: mode 0: every finite bf16 numerator with |x| >= 2^-100 against n_divisors pseudo-random divisors
 * in [2^-60, 2^60) (seed selects them); mode 1: the same with significands of all ones; mode 2: every float below
 * 2^23 in magnitude through the rounding (n_divisors, seed ignored).  out_dev: device uint64[1], receives the number
 * of mismatches (0 expected).  Asynchronous on stream. */
da2_status_t da2_selfcheck_quantiser_arithmetic(int32_t mode, int32_t n_divisors, uint32_t seed, void *out_dev,
                                                void *stream);

/* Tensor-core microbenchmark (diagnostic; the paper has no counterpart).  Every one of `ctas` CTAs issues
 * 4*iters back-to-back tcgen05.mma instructions of one kind with M = 128 and the given N (64, 128 or 256), operands
 * in shared memory, accumulators in tensor memory.  kind: 0 bf16 (K = 16 per instruction), 1 INT8 (K = 32),
 * 2 E4M3 (K = 32), 3 block-scaled NVFP4 (K = 64).  out_dev: DEVICE int64[4]: [0] clock cycles CTA 0 needed,
 * [1] instructions it issued, [2] non-zero if its bounded wait for completion gave up.  Flops per instruction are
 * 2*128*N*K.  Enqueues on stream; time the launch with events for a whole-GPU figure. */
da2_status_t da2_tcgen05_peak(int32_t kind, int32_t n, int32_t iters, int32_t ctas, void *out_dev, void *stream);

/*
 * Draft attention map without any device allocation or caller workspace (the paper has no counterpart: this is a
 * packaging variant of the draft-map step for callers that cannot allocate).
 *
 * Who needs it: code that must not call cudaMalloc -- e.g. a serving loop where an allocation would stall the device,
 * or a component whose device memory is owned and fully handed out by someone else -- and therefore cannot provide
 * the workspace da2_prepare wants.  The scratch for the two branches' draft logits lives in a fixed device array
 * inside the library (8 MiB, held by every GPU that loads the library until the process exits).
 *
 *   q_avg, q_max, k_avg, k_max : DEVICE, fp32 [BH][R][head_dim], 16-byte aligned (region descriptors, inputs)
 *   map_out                    : DEVICE, fp32 [BH][R][R] (output, rows sum to 1)
 *   limit                      : BH*R*R <= 1,048,576 and R <= 16384, head_dim a multiple of 16; larger problems
 *                                return DA2_ERR_WORKSPACE_TOO_SMALL and launch nothing.  BH <= 32767 (a launch
 *                                dimension): more heads return DA2_ERR_UNSUPPORTED and launch nothing
 * The first call on each device looks up the array's device address (with that device current); make that first
 * call outside any stream capture.  All calls on a device share the array, which keeps the previous call's
 * contents; every entry a call reads is written by that call first, so nothing needs clearing, but two calls whose
 * kernels overlap on the GPU (different streams, no ordering) race on it: order them.
 * Calls no cudaMalloc / cudaFree / allocating library routine.  Enqueues on stream, does not synchronise.
 */
da2_status_t da2_draft_map_noalloc(const float *q_avg, const float *q_max, const float *k_avg, const float *k_max,
                                   int32_t BH, int32_t R, int32_t head_dim, float lambda, float softmax_scale,
                                   float *map_out, void *stream);

void da2_plan_destroy(da2_plan_t *plan);
const char *da2_status_string(da2_status_t status);

#ifdef __cplusplus
}
#endif
#endif /* DA2_H_ */
