// team_route_static: the router step for callers that may not allocate device memory.
//
// The regular path keeps the router logits in a context workspace obtained with cudaMalloc.  Here the
// same two kernels run against a fixed scratch array that is part of the library image, so the call
// needs no context and performs no allocation of any kind.
#include <cstring>
#include <mutex>

#include "team_common.cuh"

namespace team {

// [TEAM_STATIC_ROUTE_MAX_ROWS][TEAM_MAX_EXPERTS] fp32 logits: 256 KiB, resident on every GPU that loads
// the library, for as long as the process lives.
static __device__ __align__(256) float g_static_logits[TEAM_STATIC_ROUTE_MAX_ROWS * TEAM_MAX_EXPERTS];

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
float* g_logits_addr[kMaxDevices] = {};   // device address of g_static_logits, per device ordinal

// Once per device, with that device current: resolve the scratch array's device address.  In host
// code the array's name is only a handle for the runtime, never something a kernel may dereference.
int setup_device(int dev, int dtype, int hidden, float** logits_out) {
  if (dev < 0 || dev >= kMaxDevices) return TEAM_ERR_ARG;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (g_logits_addr[dev] == nullptr) {
    float* p = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_logits);
    if (e != cudaSuccess || p == nullptr) {
      cudaGetLastError();
      return TEAM_ERR_CUDA;
    }
    g_logits_addr[dev] = p;
  }
  // The logits kernels need their dynamic shared memory opted in (an attribute, not an allocation;
  // a no-op once a call or a context has prepared at least this hidden size on the device).
  if (configure_router(dtype, hidden) != cudaSuccess) {
    cudaGetLastError();
    return TEAM_ERR_CUDA;
  }
  *logits_out = g_logits_addr[dev];
  return TEAM_OK;
}

}  // namespace
}  // namespace team

extern "C" int team_route_static(const team_config* cfg, const void* x, const void* w_router,
                                 const team_step_state* st, team_routing* out, void* stream) {
  if (cfg == nullptr || x == nullptr || w_router == nullptr || st == nullptr || out == nullptr) return TEAM_ERR_ARG;
  if (!st->tok_state) return TEAM_ERR_ARG;
  if (cfg->hidden <= 0 || cfg->n_experts <= 0 || cfg->top_k <= 0) return TEAM_ERR_SHAPE;
  if (cfg->n_experts > TEAM_MAX_EXPERTS || cfg->top_k > TEAM_MAX_TOPK || cfg->top_k > cfg->n_experts) return TEAM_ERR_SHAPE;
  if (cfg->dtype == TEAM_DTYPE_F32) {
    if (cfg->hidden % 4) return TEAM_ERR_SHAPE;
  } else if (cfg->dtype == TEAM_DTYPE_BF16) {
    if (cfg->hidden % 128) return TEAM_ERR_SHAPE;
  } else {
    return TEAM_ERR_SHAPE;
  }
  if (st->n_rows < 1) return TEAM_ERR_ARG;
  if (st->n_rows > TEAM_STATIC_ROUTE_MAX_ROWS) return TEAM_ERR_CAPACITY;   // the fixed scratch holds no more rows
  if (((uintptr_t)x & 15) || ((uintptr_t)w_router & 15)) return TEAM_ERR_ARG;

  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    cudaGetLastError();
    return TEAM_ERR_CUDA;
  }
  // the logits kernels stage 8 rows of fp32 activations in shared memory: a hidden size that does not fit is a
  // shape the kernels do not support, not a runtime failure
  int smem_optin = 0;
  if (cudaDeviceGetAttribute(&smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) {
    cudaGetLastError();
    return TEAM_ERR_CUDA;
  }
  if ((long long)team::router_smem_bytes(cfg->hidden) > smem_optin) return TEAM_ERR_SHAPE;
  float* logits = nullptr;
  const int rc = team::setup_device(dev, cfg->dtype, cfg->hidden, &logits);
  if (rc != TEAM_OK) return rc;

  team::Dims d;
  d.T = st->n_rows; d.H = cfg->hidden; d.E = cfg->n_experts; d.k = cfg->top_k; d.I = cfg->inter; d.ns = cfg->n_shared;
  d.G = cfg->max_groups;
  d.elo = 0; d.ehi = cfg->n_experts;
  team::Policy p;
  p.flags = (cfg->refresh_every > 0 && st->step_index % cfg->refresh_every == 0) ? (cfg->flags & ~TEAM_F_DCD) : cfg->flags; p.tau_hot = cfg->tau_hot; p.L_hot = cfg->L_hot; p.inclusive = cfg->hot_dist_inclusive;
  p.prefix_decoded = cfg->prefix_decoded; p.norm_topk = cfg->norm_topk;
  team::RoutePtrs e;
  memset(&e, 0, sizeof(e));
  e.probs = out->probs; e.topk_idx = out->topk_idx; e.topk_w = out->topk_w; e.margin = out->margin;

  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // Every computed row's logits are rewritten by the first kernel and skipped rows are never read by the
  // second, so nothing in the shared scratch has to be cleared between calls.
  cudaError_t ce = team::launch_router_logits(x, cfg->dtype, static_cast<const float*>(w_router), st->tok_state, logits,
                                              nullptr, d, p.flags, s);
  if (ce == cudaSuccess) ce = team::launch_router_topk(logits, st->tok_state, e, d, p, s);
  return ce == cudaSuccess ? TEAM_OK : TEAM_ERR_CUDA;
}
