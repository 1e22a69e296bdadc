// da2_draft_map_noalloc: the draft attention map for callers that cannot allocate device memory.
//
// The regular path keeps the two branches' draft logits in the caller's workspace.  Some callers have no workspace
// to give and no way to get one: code running inside a region where cudaMalloc is forbidden or would synchronise the
// device (a latency-critical serving loop, a callback, a process whose memory pool is owned by another component and
// already fully handed out).  For them this entry point keeps that scratch in a fixed array that is part of the
// library image, so the call itself allocates nothing -- no cudaMalloc, no cudaFree, no allocating library routine.
//
// The price: the array has a fixed, modest size (kMaxLogits floats per branch), every GPU that loads the library
// carries it until the process exits, and all calls on a device share it.
#include <mutex>

#include "da2_internal.cuh"

namespace {

constexpr long long kMaxLogits = 1ll << 20;  // B*H*R*R may not exceed this (two branches -> 8 MiB of scratch)

// Scratch of both logit branches.  In host code this name is only a handle for the runtime, not a device address:
// the address the kernels get comes from cudaGetSymbolAddress below.
static __device__ __align__(256) float g_logit_scratch[2 * kMaxLogits];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
float *g_scratch_ptr[kMaxDevices] = {};

// Device address of the scratch array on the current device; looked up once per device.
cudaError_t scratch_address(float **out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!g_scratch_ptr[dev]) {
    void *ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_logit_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_ptr[dev] = static_cast<float *>(ptr);
  }
  *out = g_scratch_ptr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" da2_status_t da2_draft_map_noalloc(const float *q_avg, const float *q_max, const float *k_avg,
                                              const float *k_max, int32_t BH, int32_t R, int32_t head_dim,
                                              float lambda, float softmax_scale, float *map_out, void *stream) {
  if (!q_avg || !q_max || !k_avg || !k_max || !map_out) return DA2_ERR_INVALID_ARG;
  if (BH < 1 || R < 1 || head_dim < 16 || head_dim % 16 != 0) return DA2_ERR_INVALID_ARG;
  if (!(lambda >= 0.0f && lambda <= 1.0f) || !(softmax_scale > 0.0f)) return DA2_ERR_INVALID_ARG;
  if (((uintptr_t)q_avg | (uintptr_t)q_max | (uintptr_t)k_avg | (uintptr_t)k_max) % 16 != 0)
    return DA2_ERR_INVALID_ARG;
  // the fixed scratch array bounds the problem size
  if ((long long)BH * R * R > kMaxLogits || R > 16384) return DA2_ERR_WORKSPACE_TOO_SMALL;
  if (BH > 32767) return DA2_ERR_UNSUPPORTED;  // heads index grid dimensions y and z of the launches below
  float *scratch = nullptr;
  if (scratch_address(&scratch) != cudaSuccess) return DA2_ERR_CUDA;

  da2::Params p = {};
  p.BH = BH; p.B = BH; p.H = 1; p.R = R; p.Rt = R; p.d = head_dim;
  p.lambda = lambda;
  p.scale = softmax_scale;
  p.desc[0] = const_cast<float *>(q_avg);
  p.desc[1] = const_cast<float *>(q_max);
  p.desc[2] = const_cast<float *>(k_avg);
  p.desc[3] = const_cast<float *>(k_max);
  p.logits[0] = scratch;                          // every entry used below is overwritten before it is read,
  p.logits[1] = scratch + (size_t)BH * R * R;     // so nothing has to start at zero
  p.map = map_out;
  int launches = 0;
  cudaStream_t st = (cudaStream_t)stream;
  if (da2::launch_draft(p, st, &launches) != cudaSuccess) return DA2_ERR_CUDA;
  if (da2::launch_map_rows(p, st, &launches) != cudaSuccess) return DA2_ERR_CUDA;
  return DA2_OK;
}
