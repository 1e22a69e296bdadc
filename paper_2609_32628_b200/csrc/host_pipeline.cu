// da2_attention_host: the whole call on HOST tensors with the PCIe copies hidden behind the kernels.
//
// Heads are independent problems (pooling, ranking, preparation and attention never mix heads), so the call is cut
// into groups of heads that flow through four streams: the host-to-device copy of group g+1, da2_prepare +
// da2_attention_fwd of group g and the device-to-host copy of group g-1 run at the same time, on two device slots
// carved out of one caller-provided arena.  Groups are small at both ends (the first copy-in and the last copy-out
// are the only transfers that nothing hides) and large in between.  Everything that computes is the C ABI above.
#include <algorithm>
#include <map>
#include <vector>

#include "da2_internal.cuh"

namespace {

std::vector<int> group_sizes(int BH, int n_groups) {
  std::vector<int> g;
  if (n_groups > 0) {
    const int n = std::min(n_groups, BH), base = BH / n, extra = BH % n;
    for (int i = 0; i < n; ++i) g.push_back(base + (i < extra));
    return g;
  }
  const int cap = std::max(1, (BH + 5) / 6);
  std::vector<int> up;
  int sum = 0;
  for (int n = 1; n < cap && 2 * (sum + n) <= BH - cap; n *= 2) { up.push_back(n); sum += n; }
  g = up;
  for (int rest = BH - 2 * sum; rest > 0;) { const int m = std::min(cap, rest); g.push_back(m); rest -= m; }
  g.insert(g.end(), up.rbegin(), up.rend());
  return g;
}

struct Layout {
  std::vector<int> groups;
  int nmax = 0;
  size_t tensor_bytes = 0, ws_bytes = 0, slot_bytes = 0, status_bytes = 0;
};

da2_status_t make_layout(const da2_config_t *cfg, int n_groups, Layout *L, std::map<int, da2_plan_t *> *plans) {
  if (!cfg || cfg->B < 1 || cfg->H < 1) return DA2_ERR_INVALID_ARG;
  const int BH = cfg->B * cfg->H;
  L->groups = group_sizes(BH, n_groups);
  L->nmax = *std::max_element(L->groups.begin(), L->groups.end());
  int first = 0;
  for (int n : L->groups) {
    if (!plans->count(n)) {
      da2_config_t c = *cfg;
      c.B = 1;
      c.H = n;
      // caller-fixed scales are per head: a plan per group size is only possible when they are derived
      if (cfg->g_q || cfg->g_k || cfg->g_v) return DA2_ERR_UNSUPPORTED;
      da2_plan_t *p = nullptr;
      const da2_status_t st = da2_plan(&c, &p);
      if (st != DA2_OK) return st;
      (*plans)[n] = p;
      L->ws_bytes = std::max<size_t>(L->ws_bytes, p->info.workspace_bytes);
    }
    first += n;
  }
  const da2_plan_info_t &I = plans->begin()->second->info;
  L->tensor_bytes = ((size_t)L->nmax * (size_t)(I.N + I.n_prefix) * I.head_dim * 2 + 255) / 256 * 256;
  L->ws_bytes = (L->ws_bytes + 255) / 256 * 256;
  L->slot_bytes = 4 * L->tensor_bytes + L->ws_bytes;
  L->status_bytes = (16 * L->groups.size() + 255) / 256 * 256;  // every group's status words, kept on the device
  return DA2_OK;
}

void destroy_plans(std::map<int, da2_plan_t *> &plans) {
  for (auto &kv : plans) da2_plan_destroy(kv.second);
}

}  // namespace

extern "C" {

da2_status_t da2_attention_host_arena_bytes(const da2_config_t *cfg, int32_t n_groups, size_t *bytes_out) {
  if (!bytes_out) return DA2_ERR_INVALID_ARG;
  Layout L;
  std::map<int, da2_plan_t *> plans;
  const da2_status_t st = make_layout(cfg, n_groups, &L, &plans);
  destroy_plans(plans);
  if (st != DA2_OK) return st;
  *bytes_out = 2 * L.slot_bytes + L.status_bytes;
  return DA2_OK;
}

da2_status_t da2_attention_host(const da2_config_t *cfg, const void *hq, const void *hk, const void *hv, void *hout,
                                void *arena, size_t arena_bytes, int32_t n_groups) {
  if (!cfg || !hq || !hk || !hv || !hout || !arena) return DA2_ERR_INVALID_ARG;
  if ((uintptr_t)arena % 256 != 0) return DA2_ERR_INVALID_ARG;
  Layout L;
  std::map<int, da2_plan_t *> plans;
  da2_status_t st = make_layout(cfg, n_groups, &L, &plans);
  if (st != DA2_OK) { destroy_plans(plans); return st; }
  if (arena_bytes < 2 * L.slot_bytes + L.status_bytes) { destroy_plans(plans); return DA2_ERR_WORKSPACE_TOO_SMALL; }
  uint8_t *dev_status = (uint8_t *)arena + 2 * L.slot_bytes;

  const da2_plan_info_t &I0 = plans.begin()->second->info;
  const size_t head_bytes = (size_t)(I0.N + I0.n_prefix) * I0.head_dim * 2;
  const int G = (int)L.groups.size();
  // one compute stream per device slot: consecutive groups share nothing, so the first kernels of group g+1 fill the
  // SMs that the last, partly filled wave of group g's attention kernel leaves idle
  cudaStream_t s_in = nullptr, s_cs[2] = {nullptr, nullptr}, s_out = nullptr;
  std::vector<cudaEvent_t> e_in(G, nullptr), e_c(G, nullptr), e_out(G, nullptr);
  std::vector<int> status(4 * (size_t)G, 0);
  bool ok = cudaStreamCreateWithFlags(&s_in, cudaStreamNonBlocking) == cudaSuccess &&
            cudaStreamCreateWithFlags(&s_cs[0], cudaStreamNonBlocking) == cudaSuccess &&
            cudaStreamCreateWithFlags(&s_cs[1], cudaStreamNonBlocking) == cudaSuccess &&
            cudaStreamCreateWithFlags(&s_out, cudaStreamNonBlocking) == cudaSuccess;
  for (int g = 0; ok && g < G; ++g)
    ok = cudaEventCreateWithFlags(&e_in[g], cudaEventDisableTiming) == cudaSuccess &&
         cudaEventCreateWithFlags(&e_c[g], cudaEventDisableTiming) == cudaSuccess &&
         cudaEventCreateWithFlags(&e_out[g], cudaEventDisableTiming) == cudaSuccess;
  st = ok ? DA2_OK : DA2_ERR_CUDA;

  int first = 0;
  for (int g = 0; st == DA2_OK && g < G; ++g) {
    const int n = L.groups[g];
    uint8_t *slot = (uint8_t *)arena + (size_t)(g & 1) * L.slot_bytes;
    uint8_t *dq = slot, *dk = slot + L.tensor_bytes, *dv = slot + 2 * L.tensor_bytes, *dout = slot + 3 * L.tensor_bytes;
    uint8_t *ws = slot + 4 * L.tensor_bytes;
    const size_t off = (size_t)first * head_bytes, bytes = (size_t)n * head_bytes;
    da2_plan_t *plan = plans[n];
    cudaStream_t s_c = s_cs[g & 1];
    ok = true;
    if (g >= 2) ok = cudaStreamWaitEvent(s_in, e_c[g - 2], 0) == cudaSuccess;  // the slot's inputs were consumed
    ok = ok && cudaMemcpyAsync(dq, (const uint8_t *)hq + off, bytes, cudaMemcpyHostToDevice, s_in) == cudaSuccess &&
         cudaMemcpyAsync(dk, (const uint8_t *)hk + off, bytes, cudaMemcpyHostToDevice, s_in) == cudaSuccess &&
         cudaMemcpyAsync(dv, (const uint8_t *)hv + off, bytes, cudaMemcpyHostToDevice, s_in) == cudaSuccess &&
         cudaEventRecord(e_in[g], s_in) == cudaSuccess && cudaStreamWaitEvent(s_c, e_in[g], 0) == cudaSuccess;
    if (ok && g >= 2) ok = cudaStreamWaitEvent(s_c, e_out[g - 2], 0) == cudaSuccess;  // its output left the device
    if (!ok) { st = DA2_ERR_CUDA; break; }
    st = da2_prepare(plan, dq, dk, dv, ws, L.ws_bytes, s_c);
    if (st == DA2_OK) st = da2_attention_fwd(plan, dq, dk, dv, ws, dout, s_c);
    if (st != DA2_OK) break;
    // (a copy to pageable host memory here would block the host and with it the pipeline)
    ok = cudaMemcpyAsync(dev_status + 16 * (size_t)g, ws + plan->info.off_status, 16, cudaMemcpyDeviceToDevice,
                         s_c) == cudaSuccess &&
         cudaEventRecord(e_c[g], s_c) == cudaSuccess && cudaStreamWaitEvent(s_out, e_c[g], 0) == cudaSuccess &&
         cudaMemcpyAsync((uint8_t *)hout + off, dout, bytes, cudaMemcpyDeviceToHost, s_out) == cudaSuccess &&
         cudaEventRecord(e_out[g], s_out) == cudaSuccess;
    if (!ok) { st = DA2_ERR_CUDA; break; }
    first += n;
  }
  // the call is synchronous: everything enqueued above has finished when it returns
  for (cudaStream_t s : {s_in, s_cs[0], s_cs[1], s_out})
    if (s && cudaStreamSynchronize(s) != cudaSuccess && st == DA2_OK) st = DA2_ERR_CUDA;
  if (st == DA2_OK && cudaMemcpy(status.data(), dev_status, 16 * (size_t)G, cudaMemcpyDeviceToHost) != cudaSuccess)
    st = DA2_ERR_CUDA;
  if (st == DA2_OK)
    for (int g = 0; g < G; ++g) {
      const int word = status[4 * (size_t)g];
      if (word == da2::kDevTimeout) st = DA2_ERR_TIMEOUT;
      else if (word != da2::kDevOk && st == DA2_OK) st = DA2_ERR_INTERNAL;
    }
  for (int g = 0; g < G; ++g) {
    if (e_in[g]) cudaEventDestroy(e_in[g]);
    if (e_c[g]) cudaEventDestroy(e_c[g]);
    if (e_out[g]) cudaEventDestroy(e_out[g]);
  }
  for (cudaStream_t s : {s_in, s_cs[0], s_cs[1], s_out})
    if (s) cudaStreamDestroy(s);
  destroy_plans(plans);
  return st;
}

}  // extern "C"
