// C ABI of the TEAM MoE-layer library: context, argument checks, kernel launch sequences.
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "team_common.cuh"

struct team_ctx {
  team_config cfg;
  team::Workspace ws;
  void* ws_base;
  size_t ws_bytes;
  team_weights w;
  bool has_weights;
  int device;
  int n_sms;
  int item_tile;
  int last_launches;
  int force_simt;
  bool stream_path;   // bf16: the weight-streaming expert kernel runs this context's calls (else the tensor-memory kernels)
  bool can_stream, can_tile;   // what the shape allows
  int prefer;         // diagnostic knob: 0 = choose by max_rows, 1 = streaming kernel, 2 = tensor-memory kernels
  int stream_item_tile, tile_item_tile;
  bool fused_ok;      // at most 8 rows: the whole step can run as one kernel (router and selection in its prologue)
  int no_fuse;        // diagnostic knob: keep the three-kernel sequence
  int extra_arrivals; // diagnostic knob: arrivals the fused step's barrier waits for beyond the grid's own
  long long spin_cycles;   // limit of device-side waits, in SM clock cycles
  float* ordered;          // ordered combine of the one-kernel step: [SMs][max_rows][H] partial outputs (null: off)
  void* simt_act;   // diagnostic fp32-FMA path on bf16 weights: activation scratch
  // team_moe_forward_host: one device block and its pinned host mirror, [inputs | y]
  unsigned char* hs_dev;
  unsigned char* hs_pin;
  size_t hs_in_bytes, hs_y_off, hs_bytes;
  // ... and the step (copy in, kernels, copy out) recorded once as a graph, replayed while nothing it bakes in changes
  cudaGraphExec_t hs_graph;
  int hs_graph_rows;
  int hs_graph_launches;   // kernels in the recorded step
  int hs_graph_flags;      // flags of the recorded step (a refresh step runs with other flags)
  bool hs_graph_off;     // recording failed once: plain launches from then on
  char cuda_err[256];
  // expert-kernel timing
  bool timing;
  std::vector<cudaEvent_t> ev;   // pairs
  size_t ev_used;
};

namespace {

int fail_cuda(team_ctx* ctx, cudaError_t e, const char* what) {
  if (ctx) snprintf(ctx->cuda_err, sizeof(ctx->cuda_err), "%s: %s", what, cudaGetErrorString(e));
  return TEAM_ERR_CUDA;
}

team::Dims dims_of(const team_config& c, int T) {
  team::Dims d;
  d.T = T; d.H = c.hidden; d.E = c.n_experts; d.k = c.top_k; d.I = c.inter; d.ns = c.n_shared; d.G = c.max_groups;
  const int world = c.ep_world > 1 ? c.ep_world : 1, per = c.n_experts / world;
  d.elo = world > 1 ? c.ep_rank * per : 0;
  d.ehi = world > 1 ? d.elo + per : c.n_experts;
  return d;
}

// Sec. 4.1 / Table 3: on a refresh step every token is recomputed -- cached tokens count as newly accepted, which
// is what the kernels do when delayed caching is off for that call.
int step_flags(const team_config& c, const team_step_state* st) {
  const bool refresh = c.refresh_every > 0 && st != nullptr && st->step_index % c.refresh_every == 0;
  return refresh ? (c.flags & ~TEAM_F_DCD) : c.flags;
}

team::Policy policy_of(const team_config& c, const team_step_state* st) {
  team::Policy p;
  p.flags = step_flags(c, st); p.tau_hot = c.tau_hot; p.L_hot = c.L_hot; p.inclusive = c.hot_dist_inclusive;
  p.prefix_decoded = c.prefix_decoded; p.norm_topk = c.norm_topk;
  return p;
}

int check_config(const team_config* c) {
  if (c == nullptr) return TEAM_ERR_ARG;
  if (c->hidden <= 0 || c->n_experts <= 0 || c->top_k <= 0 || c->inter <= 0 || c->n_shared < 0) return TEAM_ERR_SHAPE;
  if (c->n_experts > TEAM_MAX_EXPERTS || c->top_k > TEAM_MAX_TOPK || c->top_k > c->n_experts) return TEAM_ERR_SHAPE;
  if (c->n_shared > TEAM_MAX_SHARED) return TEAM_ERR_SHAPE;
  if (c->max_rows <= 0 || c->max_rows > TEAM_MAX_ROWS) return TEAM_ERR_SHAPE;
  if (c->max_groups <= 0 || c->max_groups > TEAM_MAX_GROUPS) return TEAM_ERR_SHAPE;
  if (c->dtype == TEAM_DTYPE_F32) {
    if (c->hidden % 4 || c->inter % 16) return TEAM_ERR_SHAPE;
  } else if (c->dtype == TEAM_DTYPE_BF16) {
    if (c->hidden % 128 || c->inter % 64) return TEAM_ERR_SHAPE;
  } else {
    return TEAM_ERR_SHAPE;
  }
  if (c->L_hot < 0 || c->refresh_every < 0) return TEAM_ERR_ARG;
  if (c->ep_world > 1) {
    if (c->ep_rank < 0 || c->ep_rank >= c->ep_world) return TEAM_ERR_ARG;
    if (c->n_experts % c->ep_world || c->n_shared != 0 || c->n_experts / c->ep_world < 1) return TEAM_ERR_SHAPE;
  }
  return TEAM_OK;
}

int check_state(const team_ctx* ctx, const team_step_state* st) {
  if (ctx == nullptr || st == nullptr) return TEAM_ERR_ARG;
  if (st->n_rows < 1 || st->n_rows > ctx->cfg.max_rows) return TEAM_ERR_ARG;
  if (!st->tok_state || !st->conf || !st->pos || !st->group || !st->branch) return TEAM_ERR_ARG;
  return TEAM_OK;
}

team::StepPtrs step_ptrs(const team_step_state* st) {
  team::StepPtrs s;
  s.tok_state = st->tok_state; s.conf = st->conf; s.pos = st->pos; s.group = st->group; s.branch = st->branch;
  return s;
}

team::RoutePtrs export_ptrs(const team_routing* r) {
  team::RoutePtrs e;
  memset(&e, 0, sizeof(e));
  if (r == nullptr) return e;
  e.probs = r->probs; e.topk_idx = r->topk_idx; e.topk_w = r->topk_w; e.margin = r->margin;
  e.tok_class = r->tok_class; e.group_mask = r->group_mask; e.expert_count = r->expert_count;
  e.expert_offset = r->expert_offset; e.perm = r->perm; e.active = r->active; e.n_active = r->n_active;
  e.n_rows_active = r->n_rows_active;
  return e;
}

// Weight pointers, policy and kernel choice are baked into the recorded host-buffer step.
void drop_host_graph(team_ctx* ctx) {
  if (ctx->hs_graph) cudaGraphExecDestroy(ctx->hs_graph);
  ctx->hs_graph = nullptr;
  ctx->hs_graph_rows = 0;
}

// Expert parallelism: the context holds its own experts' weights only; the kernels index experts by their global
// id, so every expert-weight pointer is moved back by the first local expert's offset (plain address arithmetic:
// the kernels only ever touch the experts of the local range).
const void* expert_base(const void* p, const team_ctx* ctx, const team::Dims& d) {
  if (p == nullptr || d.elo == 0) return p;
  const size_t elt = ctx->cfg.dtype == TEAM_DTYPE_F32 ? 4 : 2;
  const size_t per_expert = (size_t)d.I * d.H * elt;
  return reinterpret_cast<const void*>(reinterpret_cast<uintptr_t>(p) - (uintptr_t)d.elo * per_expert);
}

const void* gu_tiles_base(const team_ctx* ctx, const team::Dims& d) {      // gate and up tiles: two matrices per expert
  const void* p = ctx->w.w_gu_tiles;
  if (p == nullptr || d.elo == 0) return p;
  return reinterpret_cast<const void*>(reinterpret_cast<uintptr_t>(p) - (uintptr_t)d.elo * ((size_t)2 * d.I * d.H * 2));
}

// The next pair of timing events of the context (created on demand).
cudaError_t timing_events(team_ctx* ctx, cudaEvent_t* e0, cudaEvent_t* e1) {
  while (ctx->ev_used + 2 > ctx->ev.size()) {
    cudaEvent_t ne;
    const cudaError_t e = cudaEventCreate(&ne);
    if (e != cudaSuccess) return e;
    ctx->ev.push_back(ne);
  }
  *e0 = ctx->ev[ctx->ev_used];
  *e1 = ctx->ev[ctx->ev_used + 1];
  ctx->ev_used += 2;
  return cudaSuccess;
}

bool use_tensor_path(const team_ctx* ctx) { return ctx->cfg.dtype == TEAM_DTYPE_BF16 && !ctx->force_simt; }

// Calls of fewer rows than this run the weight-streaming kernel when the shape allows both (measured crossover).
constexpr int kTileMinRows = 96;

void choose_expert_kernel(team_ctx* ctx) {
  bool stream = ctx->can_stream && (!ctx->can_tile || ctx->cfg.max_rows < kTileMinRows);
  if (ctx->prefer == 1 && ctx->can_stream) stream = true;
  if (ctx->prefer == 2 && ctx->can_tile) stream = false;
  ctx->stream_path = stream;
  ctx->item_tile = stream ? ctx->stream_item_tile : ctx->tile_item_tile;
}

}  // namespace

extern "C" {

int team_version(void) { return 1; }

const char* team_strerror(int code) {
  switch (code) {
    case TEAM_OK: return "ok";
    case TEAM_ERR_ARG: return "invalid argument";
    case TEAM_ERR_SHAPE: return "unsupported shape or configuration";
    case TEAM_ERR_CUDA: return "CUDA error";
    case TEAM_ERR_TIMEOUT: return "device wait expired";
    case TEAM_ERR_STATE: return "row layout contract broken or index out of range";
    case TEAM_ERR_CAPACITY: return "more rows than the fixed-size scratch area holds";
    default: return "unknown error";
  }
}

const char* team_last_cuda_error(const team_ctx* ctx) { return ctx ? ctx->cuda_err : ""; }

int team_create(const team_config* cfg, team_ctx** out) {
  if (out == nullptr) return TEAM_ERR_ARG;
  *out = nullptr;
  int rc = check_config(cfg);
  if (rc != TEAM_OK) return rc;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0) {
    cudaGetLastError();
    return TEAM_ERR_CUDA;
  }
  team_ctx* ctx = new (std::nothrow) team_ctx();
  if (ctx == nullptr) return TEAM_ERR_ARG;
  ctx->cfg = *cfg;
  ctx->has_weights = false;
  ctx->last_launches = 0;
  ctx->force_simt = 0;
  ctx->simt_act = nullptr;
  ctx->hs_dev = nullptr;
  ctx->hs_pin = nullptr;
  ctx->hs_graph = nullptr;
  ctx->hs_graph_rows = 0;
  ctx->hs_graph_launches = 0;
  ctx->hs_graph_off = false;
  ctx->cuda_err[0] = 0;
  ctx->timing = false;
  ctx->ev_used = 0;
  ctx->fused_ok = false;
  ctx->no_fuse = 0;
  ctx->extra_arrivals = 0;
  ctx->spin_cycles = 2000000000ll;      // about a second
  ctx->ordered = nullptr;
  cudaError_t e = cudaGetDevice(&ctx->device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->n_sms, cudaDevAttrMultiProcessorCount, ctx->device);
  if (e != cudaSuccess) {
    delete ctx;
    return TEAM_ERR_CUDA;
  }
  const bool bf16 = cfg->dtype == TEAM_DTYPE_BF16;
  ctx->can_stream = bf16 && team::experts_stream_supported(cfg->max_rows, cfg->hidden, cfg->inter);
  ctx->can_tile = bf16 && team::experts_tile_supported(cfg->hidden, cfg->inter);
  if (bf16 && !ctx->can_stream && !ctx->can_tile) {
    delete ctx;
    return TEAM_ERR_SHAPE;
  }
  ctx->prefer = 0;
  // work items: the streaming kernel's gather mode takes 8 or 16 token-slots, the tensor-memory kernels up to 128
  ctx->stream_item_tile = ctx->can_stream && team::experts_stream_gathers(cfg->max_rows) ? team::experts_stream_item_tile(cfg->max_rows) : 8;
  ctx->tile_item_tile = team::experts_tile_chunk();
  choose_expert_kernel(ctx);
  e = team::configure_router(cfg->dtype, cfg->hidden);
  if (e == cudaSuccess) e = team::configure_select(dims_of(*cfg, cfg->max_rows));
  if (e == cudaSuccess && ctx->can_tile) e = team::configure_experts_tile();
  if (e == cudaSuccess && ctx->can_stream) e = team::configure_experts_stream(cfg->hidden, cfg->max_rows);
  if (e != cudaSuccess) {
    delete ctx;
    return TEAM_ERR_CUDA;
  }
  ctx->fused_ok = ctx->can_stream && team::step_fused_supported(cfg->hidden, cfg->max_rows, cfg->n_experts, ctx->n_sms);

  const size_t T = cfg->max_rows, E = cfg->n_experts, k = cfg->top_k, ns = cfg->n_shared, EN = E + ns;
  const size_t S = T * (k + ns);
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t at = off;
    off += (bytes + 255) & ~size_t(255);
    return at;
  };
  const size_t o_logits = take(T * E * 4), o_idx = take(T * k * 4), o_w = take(T * k * 4), o_margin = take(T * 4);
  const size_t o_cls = take(T), o_gm = take((size_t)cfg->max_groups * ((E + 63) / 64) * 8);
  const size_t o_cnt = take(EN * 4), o_off = take((EN + 1) * 4), o_perm = take(S * 4), o_act_list = take(EN * 4);
  const size_t o_scal = take(64), o_items = take((EN + S / 8 + 2) * sizeof(team::WorkItem));
  const size_t o_act = take(cfg->dtype == TEAM_DTYPE_F32 ? S * cfg->inter * 4 : 256);
  // the tensor-memory kernels' gathered token tiles, activation tiles and per-slot tables
  const size_t tile_items = EN + S / ctx->tile_item_tile + 2;
  const size_t tile_rows = ctx->can_tile ? team::experts_tile_rows(S, tile_items) : 0;
  const size_t o_trow = take(tile_rows * 4 + 4), o_tw = take(tile_rows * 4 + 4);
  const size_t o_tx = take(tile_rows * cfg->hidden * 2 + 256), o_tact = take(tile_rows * cfg->inter * 2 + 256);
  ctx->ws_bytes = off;
  e = cudaMalloc(&ctx->ws_base, ctx->ws_bytes);
  if (e != cudaSuccess) {
    delete ctx;
    return TEAM_ERR_CUDA;
  }
  cudaMemset(ctx->ws_base, 0, ctx->ws_bytes);
  unsigned char* b = static_cast<unsigned char*>(ctx->ws_base);
  team::Workspace& ws = ctx->ws;
  ws.logits = reinterpret_cast<float*>(b + o_logits);
  ws.r.probs = nullptr;
  ws.r.topk_idx = reinterpret_cast<int32_t*>(b + o_idx);
  ws.r.topk_w = reinterpret_cast<float*>(b + o_w);
  ws.r.margin = reinterpret_cast<float*>(b + o_margin);
  ws.r.tok_class = b + o_cls;
  ws.r.group_mask = reinterpret_cast<uint64_t*>(b + o_gm);
  ws.r.expert_count = reinterpret_cast<int32_t*>(b + o_cnt);
  ws.r.expert_offset = reinterpret_cast<int32_t*>(b + o_off);
  ws.r.perm = reinterpret_cast<int32_t*>(b + o_perm);
  ws.r.active = reinterpret_cast<int32_t*>(b + o_act_list);
  int32_t* scal = reinterpret_cast<int32_t*>(b + o_scal);
  ws.r.n_active = scal + 0;
  ws.r.n_rows_active = scal + 1;
  ws.n_items = scal + 2;
  ws.status = scal + 4;
  ws.arrivals = reinterpret_cast<unsigned long long*>(scal + 8);
  ws.items = reinterpret_cast<team::WorkItem*>(b + o_items);
  ws.act = reinterpret_cast<float*>(b + o_act);
  ws.tile_row = reinterpret_cast<int32_t*>(b + o_trow);
  ws.tile_w = reinterpret_cast<float*>(b + o_tw);
  ws.tile_x = reinterpret_cast<__nv_bfloat16*>(b + o_tx);
  ws.tile_act = reinterpret_cast<__nv_bfloat16*>(b + o_tact);
  *out = ctx;
  return TEAM_OK;
}

int team_destroy(team_ctx* ctx) {
  if (ctx == nullptr) return TEAM_ERR_ARG;
  for (cudaEvent_t e : ctx->ev) cudaEventDestroy(e);
  cudaFree(ctx->ws_base);
  if (ctx->simt_act) cudaFree(ctx->simt_act);
  if (ctx->ordered) cudaFree(ctx->ordered);
  if (ctx->hs_dev) cudaFree(ctx->hs_dev);
  if (ctx->hs_pin) cudaFreeHost(ctx->hs_pin);
  if (ctx->hs_graph) cudaGraphExecDestroy(ctx->hs_graph);
  delete ctx;
  return TEAM_OK;
}

int team_set_weights(team_ctx* ctx, const team_weights* w) {
  if (ctx == nullptr || w == nullptr) return TEAM_ERR_ARG;
  if (!w->w_router || ((uintptr_t)w->w_router & 15)) return TEAM_ERR_ARG;
  // expert weights: the row-major / slab set, the tile-major set, or both; each set is all or nothing
  const bool classic = w->w_gate || w->w_up || w->w_down, tiles = w->w_gu_tiles || w->w_down_tiles;
  if (classic && !(w->w_gate && w->w_up && w->w_down)) return TEAM_ERR_ARG;
  if (tiles && !(w->w_gu_tiles && w->w_down_tiles)) return TEAM_ERR_ARG;
  if (!classic && !tiles) return TEAM_ERR_ARG;
  const uintptr_t align = ctx->cfg.dtype == TEAM_DTYPE_BF16 ? 127 : 15;
  if (classic && (((uintptr_t)w->w_gate & align) || ((uintptr_t)w->w_up & align) || ((uintptr_t)w->w_down & align)))
    return TEAM_ERR_ARG;
  if (tiles && (((uintptr_t)w->w_gu_tiles & 127) || ((uintptr_t)w->w_down_tiles & 127))) return TEAM_ERR_ARG;
  if (tiles && ctx->cfg.dtype != TEAM_DTYPE_BF16) return TEAM_ERR_ARG;
  ctx->w = *w;
  ctx->has_weights = true;
  drop_host_graph(ctx);
  return TEAM_OK;
}

int team_set_policy(team_ctx* ctx, const team_config* cfg) {
  if (ctx == nullptr || cfg == nullptr) return TEAM_ERR_ARG;
  const team_config& c = ctx->cfg;
  if (cfg->hidden != c.hidden || cfg->n_experts != c.n_experts || cfg->top_k != c.top_k || cfg->inter != c.inter ||
      cfg->n_shared != c.n_shared || cfg->max_rows != c.max_rows || cfg->max_groups != c.max_groups ||
      cfg->dtype != c.dtype || cfg->ep_rank != c.ep_rank || cfg->ep_world != c.ep_world)
    return TEAM_ERR_SHAPE;
  if (cfg->L_hot < 0 || cfg->refresh_every < 0) return TEAM_ERR_ARG;
  ctx->cfg = *cfg;
  drop_host_graph(ctx);
  return TEAM_OK;
}

int team_debug_force_simt(team_ctx* ctx, int on) {
  if (ctx == nullptr) return TEAM_ERR_ARG;
  if (on && ctx->cfg.dtype == TEAM_DTYPE_BF16 && ctx->simt_act == nullptr) {
    const size_t S = (size_t)ctx->cfg.max_rows * (ctx->cfg.top_k + ctx->cfg.n_shared);
    cudaError_t e = cudaMalloc(&ctx->simt_act, S * ctx->cfg.inter * 4);
    if (e != cudaSuccess) return fail_cuda(ctx, e, "diagnostic scratch");
    ctx->ws.act = static_cast<float*>(ctx->simt_act);
  }
  ctx->force_simt = on;
  drop_host_graph(ctx);
  return TEAM_OK;
}

int team_route(team_ctx* ctx, const void* x, const team_step_state* st, team_routing* out, void* stream) {
  int rc = check_state(ctx, st);
  if (rc != TEAM_OK) return rc;
  if (x == nullptr || out == nullptr || !ctx->has_weights) return TEAM_ERR_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const team::Dims d = dims_of(ctx->cfg, st->n_rows);
  ctx->last_launches = 0;
  cudaError_t e = team::launch_router_logits(x, ctx->cfg.dtype, static_cast<const float*>(ctx->w.w_router),
                                             st->tok_state, ctx->ws.logits, nullptr, d, step_flags(ctx->cfg, st), s);
  if (e != cudaSuccess) return fail_cuda(ctx, e, "router logits");
  ++ctx->last_launches;
  e = team::launch_router_topk(ctx->ws.logits, st->tok_state, export_ptrs(out), d, policy_of(ctx->cfg, st), s);
  if (e != cudaSuccess) return fail_cuda(ctx, e, "router top-k");
  ++ctx->last_launches;
  return TEAM_OK;
}

int team_select_experts(team_ctx* ctx, const team_step_state* st, team_routing* out, void* stream) {
  int rc = check_state(ctx, st);
  if (rc != TEAM_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const team::Dims d = dims_of(ctx->cfg, st->n_rows);
  ctx->last_launches = 0;
  cudaError_t e = team::launch_select(ctx->ws.logits, step_ptrs(st), ctx->ws, export_ptrs(out), d,
                                      policy_of(ctx->cfg, st), ctx->item_tile, true, s);
  if (e != cudaSuccess) return fail_cuda(ctx, e, "select");
  ctx->last_launches += team::select_launches(d);
  return TEAM_OK;
}

int team_moe_forward(team_ctx* ctx, const void* x, const team_step_state* st, team_routing* out, float* y,
                     void* stream) {
  int rc = check_state(ctx, st);
  if (rc != TEAM_OK) return rc;
  if (x == nullptr || y == nullptr || !ctx->has_weights) return TEAM_ERR_ARG;
  if (((uintptr_t)x & 15) || ((uintptr_t)y & 15)) return TEAM_ERR_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const team::Dims d = dims_of(ctx->cfg, st->n_rows);
  const bool tc = use_tensor_path(ctx);
  ctx->last_launches = 0;
  // the weight layout the expert kernel of this context reads must have been given
  if (tc && ctx->stream_path && !ctx->w.w_gate) return TEAM_ERR_ARG;
  if (tc && !ctx->stream_path && !ctx->w.w_gu_tiles) return TEAM_ERR_ARG;
  if (!tc && !ctx->w.w_gate) return TEAM_ERR_ARG;
  // The resident few-rows expert kernel reads the rows' choices directly; the dispatch tables are built only
  // when the caller asked for one of them.
  const bool wants_tables = out != nullptr && (out->expert_count || out->expert_offset || out->perm || out->active ||
                                               out->n_active || out->n_rows_active);
  const bool resident = tc && ctx->stream_path && !team::experts_stream_gathers(ctx->cfg.max_rows);
  cudaError_t e = cudaSuccess;
  cudaEvent_t ev0 = nullptr, ev1 = nullptr;
  if (resident && !wants_tables && ctx->fused_ok && !ctx->no_fuse) {
    // at most 8 rows and no dispatch table asked for: the whole step is one kernel
    if (ctx->timing && (e = timing_events(ctx, &ev0, &ev1)) != cudaSuccess) return fail_cuda(ctx, e, "event create");
    if (ev0) cudaEventRecord(ev0, s);
    e = team::launch_step_fused(x, static_cast<const float*>(ctx->w.w_router), expert_base(ctx->w.w_gate, ctx, d),
                                expert_base(ctx->w.w_up, ctx, d), expert_base(ctx->w.w_down, ctx, d),
                                step_ptrs(st), ctx->ws, export_ptrs(out), y, d, policy_of(ctx->cfg, st), ctx->n_sms,
                                ctx->spin_cycles, ctx->extra_arrivals, ctx->ordered, s);
    if (e != cudaSuccess) return fail_cuda(ctx, e, "fused step");
    if (ev1) cudaEventRecord(ev1, s);
    ctx->last_launches = 1;
    return TEAM_OK;
  }
  e = team::launch_router_logits(x, ctx->cfg.dtype, static_cast<const float*>(ctx->w.w_router), st->tok_state,
                                 ctx->ws.logits, tc ? y : nullptr, d, step_flags(ctx->cfg, st), s);
  if (e != cudaSuccess) return fail_cuda(ctx, e, "router logits");
  ++ctx->last_launches;
  e = team::launch_select(ctx->ws.logits, step_ptrs(st), ctx->ws, export_ptrs(out), d, policy_of(ctx->cfg, st),
                          ctx->item_tile, wants_tables || !resident, s);
  if (e != cudaSuccess) return fail_cuda(ctx, e, "select");
  ctx->last_launches += team::select_launches(d);
  if (ctx->timing) {
    if ((e = timing_events(ctx, &ev0, &ev1)) != cudaSuccess) return fail_cuda(ctx, e, "event create");
    cudaEventRecord(ev0, s);
  }
  if (tc) {
    if (ctx->stream_path)
      e = team::launch_experts_stream(x, expert_base(ctx->w.w_gate, ctx, d), expert_base(ctx->w.w_up, ctx, d),
                                      expert_base(ctx->w.w_down, ctx, d), ctx->ws, y, d, ctx->cfg.max_rows, ctx->n_sms, s);
    else
      e = team::launch_experts_tile(x, gu_tiles_base(ctx, d), expert_base(ctx->w.w_down_tiles, ctx, d), ctx->ws, y, d,
                                    ctx->n_sms, s);
    if (e != cudaSuccess) return fail_cuda(ctx, e, "expert kernel");
    ctx->last_launches += ctx->stream_path ? 1 : 3;
  } else {
    e = team::launch_experts_simt(x, ctx->cfg.dtype, expert_base(ctx->w.w_gate, ctx, d), expert_base(ctx->w.w_up, ctx, d),
                                  expert_base(ctx->w.w_down, ctx, d), ctx->ws, y, d, s);
    if (e != cudaSuccess) return fail_cuda(ctx, e, "expert kernels (fp32)");
    ctx->last_launches += 2;
  }
  if (ev1) cudaEventRecord(ev1, s);
  return TEAM_OK;
}

int team_moe_forward_host(team_ctx* ctx, const void* x_host, const team_step_state* st_host, team_routing* out,
                          float* y_host, void* stream) {
  int rc = check_state(ctx, st_host);
  if (rc != TEAM_OK) return rc;
  if (x_host == nullptr || y_host == nullptr || !ctx->has_weights) return TEAM_ERR_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t Tm = ctx->cfg.max_rows, H = ctx->cfg.hidden, elt = ctx->cfg.dtype == TEAM_DTYPE_F32 ? 4 : 2;
  auto up = [](size_t v) { return (v + 255) & ~size_t(255); };
  // layout of the staging block (sized for max_rows): x | tok_state | conf | pos | group | branch | y
  const size_t o_x = 0, o_ts = up(Tm * H * elt), o_conf = o_ts + up(Tm), o_pos = o_conf + up(Tm * 4),
               o_grp = o_pos + up(Tm * 4), o_br = o_grp + up(Tm * 4), o_y = o_br + up(Tm * 4);
  if (ctx->hs_dev == nullptr) {
    ctx->hs_in_bytes = o_y;
    ctx->hs_y_off = o_y;
    ctx->hs_bytes = o_y + up(Tm * H * 4);
    cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&ctx->hs_dev), ctx->hs_bytes);
    if (e == cudaSuccess) e = cudaMemsetAsync(ctx->hs_dev, 0, ctx->hs_bytes, s);
    if (e == cudaSuccess) e = cudaMallocHost(reinterpret_cast<void**>(&ctx->hs_pin), ctx->hs_bytes);
    if (e != cudaSuccess) {
      if (ctx->hs_dev) cudaFree(ctx->hs_dev);
      ctx->hs_dev = nullptr;
      return fail_cuda(ctx, e, "host staging");
    }
    memset(ctx->hs_pin, 0, ctx->hs_bytes);
  }
  const size_t T = st_host->n_rows;
  unsigned char* hp = ctx->hs_pin;
  memcpy(hp + o_x, x_host, T * H * elt);
  memcpy(hp + o_ts, st_host->tok_state, T);
  memcpy(hp + o_conf, st_host->conf, T * 4);
  memcpy(hp + o_pos, st_host->pos, T * 4);
  memcpy(hp + o_grp, st_host->group, T * 4);
  memcpy(hp + o_br, st_host->branch, T * 4);
  // one copy in: with few rows the block is small and a single transfer beats six
  const size_t in_bytes = ctx->hs_in_bytes;
  unsigned char* dp = ctx->hs_dev;
  team_step_state st = *st_host;
  st.tok_state = dp + o_ts;
  st.conf = reinterpret_cast<const float*>(dp + o_conf);
  st.pos = reinterpret_cast<const int32_t*>(dp + o_pos);
  st.group = reinterpret_cast<const int32_t*>(dp + o_grp);
  st.branch = reinterpret_cast<const int32_t*>(dp + o_br);
  float* y_dev = reinterpret_cast<float*>(dp + ctx->hs_y_off);
  // copy in, the layer, copy out: all addresses are the context's own, so the sequence is the same every step
  auto issue = [&]() -> int {
    cudaError_t e = cudaMemcpyAsync(ctx->hs_dev, hp, in_bytes, cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return fail_cuda(ctx, e, "copy in");
    const int r = team_moe_forward(ctx, dp + o_x, &st, out, y_dev, stream);
    if (r != TEAM_OK) return r;
    e = cudaMemcpyAsync(hp + ctx->hs_y_off, y_dev, T * H * 4, cudaMemcpyDeviceToHost, s);
    return e == cudaSuccess ? TEAM_OK : fail_cuda(ctx, e, "copy out");
  };
  // Replayed as one graph launch when possible: a stream that can be captured (not the legacy default stream,
  // not already capturing), no exports, no expert timing.
  bool replay = !ctx->hs_graph_off && s != nullptr && s != cudaStreamLegacy && out == nullptr && !ctx->timing;
  if (replay) {
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(s, &cap) != cudaSuccess || cap != cudaStreamCaptureStatusNone) {
      cudaGetLastError();
      replay = false;
    }
  }
  if (replay && (ctx->hs_graph == nullptr || ctx->hs_graph_rows != (int)T || ctx->hs_graph_flags != step_flags(ctx->cfg, st_host))) {
    drop_host_graph(ctx);
    cudaGraph_t g = nullptr;
    bool good = cudaStreamBeginCapture(s, cudaStreamCaptureModeThreadLocal) == cudaSuccess;
    if (good) {
      const int r = issue();
      const cudaError_t e = cudaStreamEndCapture(s, &g);
      good = r == TEAM_OK && e == cudaSuccess && g != nullptr;
    }
    if (good) good = cudaGraphInstantiate(&ctx->hs_graph, g, 0) == cudaSuccess;
    if (g) cudaGraphDestroy(g);
    if (good) {
      ctx->hs_graph_rows = (int)T;
      ctx->hs_graph_launches = ctx->last_launches;
      ctx->hs_graph_flags = step_flags(ctx->cfg, st_host);
    } else {
      cudaGetLastError();
      ctx->hs_graph = nullptr;
      ctx->hs_graph_off = true;
      replay = false;
    }
  }
  if (replay) {
    const cudaError_t e = cudaGraphLaunch(ctx->hs_graph, s);
    if (e != cudaSuccess) return fail_cuda(ctx, e, "graph launch");
    ctx->last_launches = ctx->hs_graph_launches;
  } else {
    rc = issue();
    if (rc != TEAM_OK) return rc;
  }
  const cudaError_t es = cudaStreamSynchronize(s);
  if (es != cudaSuccess) return fail_cuda(ctx, es, "synchronise");
  memcpy(y_host, hp + ctx->hs_y_off, T * H * 4);
  return TEAM_OK;
}

int team_residual_add(team_ctx* ctx, void* x, const float* y, int32_t n_rows, void* stream) {
  if (ctx == nullptr || x == nullptr || y == nullptr || n_rows < 1 || n_rows > ctx->cfg.max_rows) return TEAM_ERR_ARG;
  cudaError_t e = team::launch_residual_add(x, ctx->cfg.dtype, y, ctx->ws.r.tok_class, n_rows, ctx->cfg.hidden,
                                            static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return fail_cuda(ctx, e, "residual add");
  ctx->last_launches = 1;
  return TEAM_OK;
}

int team_read_status(team_ctx* ctx, void* stream, int32_t* detail_out) {
  if (ctx == nullptr) return TEAM_ERR_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int32_t host[2] = {0, 0};
  cudaError_t e = cudaMemcpyAsync(host, ctx->ws.status, sizeof(host), cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaMemsetAsync(ctx->ws.status, 0, sizeof(host), s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return fail_cuda(ctx, e, "read status");
  if (detail_out) *detail_out = host[1];
  return host[0];
}

int team_last_launch_count(const team_ctx* ctx) { return ctx ? ctx->last_launches : 0; }

const char* team_expert_kernel_name(const team_ctx* ctx) {
  if (ctx == nullptr) return "";
  if (!use_tensor_path(ctx)) return "k_gate_up + k_down";
  if (!ctx->stream_path) return "k_grouped_gemm (tcgen05: gate/up + SwiGLU, then down + combine)";
  const bool fused = ctx->fused_ok && !ctx->no_fuse && !team::experts_stream_gathers(ctx->cfg.max_rows);
  return fused ? "k_experts_stream (fused step: router, selection and experts in one launch)" : "k_experts_stream";
}

int team_debug_knob(team_ctx* ctx, int knob, long long value) {
  if (ctx == nullptr) return TEAM_ERR_ARG;
  switch (knob) {
    case TEAM_KNOB_NO_FUSE: ctx->no_fuse = value != 0; break;
    case TEAM_KNOB_ORDERED_COMBINE:
      // only the one-kernel step has the ordered mode (its CTAs meet at a grid barrier anyway)
      if (!ctx->fused_ok || team::experts_stream_gathers(ctx->cfg.max_rows)) return TEAM_ERR_SHAPE;
      if (value != 0 && ctx->ordered == nullptr) {
        const cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&ctx->ordered),
                                         (size_t)ctx->n_sms * ctx->cfg.max_rows * ctx->cfg.hidden * sizeof(float));
        if (e != cudaSuccess) return fail_cuda(ctx, e, "ordered-combine scratch");
      } else if (value == 0 && ctx->ordered != nullptr) {
        cudaFree(ctx->ordered);
        ctx->ordered = nullptr;
      }
      break;
    case TEAM_KNOB_EXPERT_KERNEL:
      if (value < 0 || value > 2) return TEAM_ERR_ARG;
      ctx->prefer = (int)value;
      choose_expert_kernel(ctx);
      break;
    case TEAM_KNOB_EXTRA_ARRIVALS:
      if (value < 0 || value > 1) return TEAM_ERR_ARG;
      ctx->extra_arrivals = (int)value;
      break;
    case TEAM_KNOB_WAIT_LIMIT_US:
      if (value < 1 || value > 10000000) return TEAM_ERR_ARG;
      ctx->spin_cycles = value * 2000;       // SM cycles at about 2 GHz
      break;
    default: return TEAM_ERR_ARG;
  }
  drop_host_graph(ctx);
  return TEAM_OK;
}

int team_expert_timing(team_ctx* ctx, int32_t enable, void* stream, float* avg_ms_out, int32_t* launches_out) {
  if (ctx == nullptr) return TEAM_ERR_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return fail_cuda(ctx, e, "timing sync");
  double total = 0.0;
  const int n = (int)(ctx->ev_used / 2);
  for (int i = 0; i < n; ++i) {
    float ms = 0.f;
    if ((e = cudaEventElapsedTime(&ms, ctx->ev[2 * i], ctx->ev[2 * i + 1])) != cudaSuccess)
      return fail_cuda(ctx, e, "event elapsed");
    total += ms;
  }
  if (avg_ms_out) *avg_ms_out = n > 0 ? (float)(total / n) : 0.f;
  if (launches_out) *launches_out = n;
  ctx->ev_used = 0;
  ctx->timing = enable != 0;
  return TEAM_OK;
}

}  // extern "C"
