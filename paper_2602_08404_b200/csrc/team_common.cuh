// Shared declarations of the TEAM MoE-layer kernels (device-side structs, small helpers).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "team.h"

namespace team {

// Shapes of one call.
struct Dims {
  int T;   // rows presented
  int H;   // hidden
  int E;   // routed experts
  int k;   // top-k
  int I;   // expert intermediate
  int ns;  // shared experts
  int G;   // max groups
  int elo, ehi;   // expert parallelism: this call computes the routed experts [elo, ehi) only (0, E without it)
};

// Eq. 4 / Algorithm 1 policy knobs.
struct Policy {
  int flags;
  float tau_hot;
  int L_hot;
  int inclusive;
  int prefix_decoded;
  int norm_topk;
};

// Previous-step state (device pointers).
struct StepPtrs {
  const uint8_t* tok_state;
  const float* conf;
  const int32_t* pos;
  const int32_t* group;
  const int32_t* branch;
};

// Routing tables.  `ws` pointers are never null; `ex` (caller exports) may be.
struct RoutePtrs {
  float* probs;
  int32_t* topk_idx;
  float* topk_w;
  float* margin;
  uint8_t* tok_class;
  uint64_t* group_mask;
  int32_t* expert_count;
  int32_t* expert_offset;
  int32_t* perm;
  int32_t* active;
  int32_t* n_active;
  int32_t* n_rows_active;
};

// One unit of expert work: `n` consecutive entries of perm starting at `begin`, all of expert `e`.
struct WorkItem {
  int32_t e;
  int32_t begin;
  int32_t n;
  int32_t pad;
};

struct Workspace {
  float* logits;        // [max_rows, E]
  RoutePtrs r;          // context-owned routing tables (probs is null here)
  WorkItem* items;      // [E + ns + max_rows*(k+ns)/tile + 1]
  int32_t* n_items;     // [1]
  float* act;           // fp32 path: [max_rows*(k+ns), I] SwiGLU activations
  int32_t* status;      // [2] code, detail
  // tensor-memory expert kernels: gathered token tiles, SwiGLU activation tiles, per-slot (row, weight) tables
  __nv_bfloat16* tile_x;    // [padded slot rows][H] as per-chunk [kb][rows][64] tiles
  __nv_bfloat16* tile_act;  // [padded slot rows][I] likewise
  int32_t* tile_row;        // [padded slot rows]
  float* tile_w;            // [padded slot rows]
  unsigned long long* arrivals;   // fused step: CTA arrivals at the grid barrier, counted over all launches
};

__device__ __forceinline__ void set_status(int32_t* status, int code, int detail) {
  if (atomicCAS(status, 0, code) == 0) status[1] = detail;
}

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }

// Row and combine weight of a slot id (routed: t*k+j, shared: T*k + s*T + t).
__device__ __forceinline__ void slot_row_weight(int slot, int T, int k, const float* topk_w, int& row, float& w) {
  if (slot < T * k) {
    row = slot / k;
    w = topk_w[slot];
  } else {
    row = (slot - T * k) % T;
    w = 1.0f;
  }
}

// Kernel launchers (host side), one per translation unit.
cudaError_t configure_router(int dtype, int hidden);
int router_smem_bytes(int hidden);   // dynamic shared memory the logits kernels are opted in to for this hidden size
cudaError_t configure_select(Dims max_dims);
bool experts_tile_supported(int hidden, int inter);
int experts_tile_chunk();
size_t experts_tile_rows(size_t slots, size_t max_items);
cudaError_t configure_experts_tile();
cudaError_t launch_experts_tile(const void* x, const void* gu_tiles, const void* d_tiles, Workspace ws, float* y, Dims d,
                                int grid, cudaStream_t s);
cudaError_t launch_pack_w_tiles(const void* w_gate, const void* w_up, const void* w_down, void* gu, void* dt, int n_exp,
                                int H, int I, cudaStream_t s);
bool experts_stream_supported(int max_rows, int hidden, int inter);
bool experts_stream_gathers(int max_rows);
int experts_stream_item_tile(int max_rows);
cudaError_t configure_experts_stream(int hidden, int max_rows);
cudaError_t launch_experts_stream(const void* x, const void* w_gate, const void* w_up, const void* w_down, Workspace ws,
                                  float* y, Dims d, int max_rows, int grid, cudaStream_t s);
bool step_fused_supported(int hidden, int max_rows, int n_experts, int grid);
cudaError_t launch_step_fused(const void* x, const float* w_router, const void* w_gate, const void* w_up, const void* w_down,
                              StepPtrs st, Workspace ws, RoutePtrs ex, float* y, Dims d, Policy p, int grid,
                              long long spin_cycles, int extra_arrivals, float* ordered, cudaStream_t s);
cudaError_t launch_router_logits(const void* x, int dtype, const float* w_router, const uint8_t* tok_state,
                                 float* logits, float* y_zero, Dims d, int flags, cudaStream_t s);
cudaError_t launch_router_topk(const float* logits, const uint8_t* tok_state, RoutePtrs out, Dims d, Policy p,
                               cudaStream_t s);
cudaError_t launch_select(const float* logits, StepPtrs st, Workspace ws, RoutePtrs ex, Dims d, Policy p,
                          int item_tile, bool need_tables, cudaStream_t s);
int select_launches(Dims d);   // kernels launch_select issues for these sizes
size_t select_smem_bytes(Dims d);
cudaError_t launch_experts_simt(const void* x, int dtype, const void* w_gate, const void* w_up, const void* w_down,
                                Workspace ws, float* y, Dims d, cudaStream_t s);
cudaError_t launch_residual_add(void* x, int dtype, const float* y, const uint8_t* tok_class, int T, int H,
                                cudaStream_t s);

}  // namespace team
