// Plain-FMA expert path (fp32 configuration, and a diagnostic path for bf16 weights).
//
//   k_gate_up : act[slot, i] = silu(W_gate[e,i,:] . x[t,:]) * (W_up[e,i,:] . x[t,:])      one warp per (slot, i)
//   k_down    : y[t, h] = sum over the row's slots of w * (W_down[e,h,:] . act[slot,:])     one warp per (t, h)
//
// Accumulation is fp32 with a fixed order (lane-strided partial sums, shuffle tree, slots in
// ascending order), so the result is deterministic; no atomics are used.  Also the stack glue.
#include "team_common.cuh"
#include "team_topk.cuh"

namespace team {

template <typename WT>
__device__ __forceinline__ float dot_row(const WT* __restrict__ w, const WT* __restrict__ v, int n, int lane);

template <>
__device__ __forceinline__ float dot_row<float>(const float* __restrict__ w, const float* __restrict__ v, int n,
                                                int lane) {
  float acc = 0.f;
  const float4* w4 = reinterpret_cast<const float4*>(w);
  const float4* v4 = reinterpret_cast<const float4*>(v);
  for (int c = lane; c < (n >> 2); c += 32) {
    const float4 a = __ldg(w4 + c), b = __ldg(v4 + c);
    acc = fmaf(a.x, b.x, acc);
    acc = fmaf(a.y, b.y, acc);
    acc = fmaf(a.z, b.z, acc);
    acc = fmaf(a.w, b.w, acc);
  }
  return warp_sum(acc);
}

template <>
__device__ __forceinline__ float dot_row<__nv_bfloat16>(const __nv_bfloat16* __restrict__ w,
                                                        const __nv_bfloat16* __restrict__ v, int n, int lane) {
  float acc = 0.f;
  const uint4* w8 = reinterpret_cast<const uint4*>(w);
  const uint4* v8 = reinterpret_cast<const uint4*>(v);
  for (int c = lane; c < (n >> 3); c += 32) {
    const uint4 a = __ldg(w8 + c), b = __ldg(v8 + c);
    const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&a);
    const __nv_bfloat162* pb = reinterpret_cast<const __nv_bfloat162*>(&b);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const float2 fa = __bfloat1622float2(pa[q]), fb = __bfloat1622float2(pb[q]);
      acc = fmaf(fa.x, fb.x, acc);
      acc = fmaf(fa.y, fb.y, acc);
    }
  }
  return warp_sum(acc);
}

// Expert and row of a slot id, or e = -1 if the slot is not computed this step.
__device__ __forceinline__ void slot_expert_row(int slot, const Dims& d, const int32_t* topk_idx,
                                                const uint8_t* tok_class, int& e, int& t) {
  if (slot < d.T * d.k) {
    t = slot / d.k;
    e = topk_idx[slot];
  } else {
    const int r = slot - d.T * d.k;
    t = r % d.T;
    e = (tok_class[t] != TEAM_CLS_SKIP) ? d.E + r / d.T : -1;
  }
}

template <typename WT>
__global__ void __launch_bounds__(256)
k_gate_up(const WT* __restrict__ x, const WT* __restrict__ w_gate, const WT* __restrict__ w_up,
          const int32_t* __restrict__ topk_idx, const uint8_t* __restrict__ tok_class, float* __restrict__ act,
          Dims d) {
  const int slot = blockIdx.y;
  int e, t;
  slot_expert_row(slot, d, topk_idx, tok_class, e, t);
  if (e < 0 || (e < d.E && (e < d.elo || e >= d.ehi))) return;      // not computed, or another rank's expert
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int i = blockIdx.x * 8 + warp;
  if (i >= d.I) return;
  const WT* xr = x + (size_t)t * d.H;
  const size_t row = ((size_t)e * d.I + i) * d.H;
  const float g = dot_row<WT>(w_gate + row, xr, d.H, lane);
  const float u = dot_row<WT>(w_up + row, xr, d.H, lane);
  if (lane == 0) act[(size_t)slot * d.I + i] = g / (1.f + expf(-g)) * u;
}

template <typename WT>
__global__ void __launch_bounds__(256)
k_down(const WT* __restrict__ w_down, const float* __restrict__ act, const int32_t* __restrict__ topk_idx,
       const float* __restrict__ topk_w, const uint8_t* __restrict__ tok_class, float* __restrict__ y, Dims d) {
  const int t = blockIdx.y;
  if (tok_class[t] == TEAM_CLS_SKIP) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int h = blockIdx.x * 8 + warp;
  if (h >= d.H) return;
  float out = 0.f;
  for (int j = 0; j < d.k + d.ns; ++j) {
    int slot, e;
    float w;
    if (j < d.k) {
      slot = t * d.k + j;
      e = topk_idx[slot];
      w = topk_w[slot];
    } else {
      slot = d.T * d.k + (j - d.k) * d.T + t;
      e = d.E + (j - d.k);
      w = 1.f;
    }
    if (e < 0 || (e < d.E && (e < d.elo || e >= d.ehi))) continue;
    // W_down is stored in slabs of 16 columns: element (e, h, c) sits at (((e * I/16 + c/16) * H + h) * 16 + c%16)
    const WT* wr = w_down + ((size_t)e * (d.I / 16) * d.H + h) * 16;
    const float* ar = act + (size_t)slot * d.I;
    float acc = 0.f;
    for (int c = lane; c < d.I; c += 32) acc = fmaf(to_f32(wr[(size_t)(c >> 4) * d.H * 16 + (c & 15)]), ar[c], acc);
    out = fmaf(w, warp_sum(acc), out);
  }
  if (lane == 0) y[(size_t)t * d.H + h] = out;
}

cudaError_t launch_experts_simt(const void* x, int dtype, const void* w_gate, const void* w_up, const void* w_down,
                                Workspace ws, float* y, Dims d, cudaStream_t s) {
  const int n_slots = d.T * (d.k + d.ns);
  dim3 g1((d.I + 7) / 8, n_slots), g2((d.H + 7) / 8, d.T);
  if (dtype == TEAM_DTYPE_F32) {
    k_gate_up<float><<<g1, 256, 0, s>>>((const float*)x, (const float*)w_gate, (const float*)w_up, ws.r.topk_idx,
                                        ws.r.tok_class, ws.act, d);
    k_down<float><<<g2, 256, 0, s>>>((const float*)w_down, ws.act, ws.r.topk_idx, ws.r.topk_w, ws.r.tok_class, y, d);
  } else {
    k_gate_up<__nv_bfloat16><<<g1, 256, 0, s>>>((const __nv_bfloat16*)x, (const __nv_bfloat16*)w_gate,
                                                (const __nv_bfloat16*)w_up, ws.r.topk_idx, ws.r.tok_class, ws.act, d);
    k_down<__nv_bfloat16><<<g2, 256, 0, s>>>((const __nv_bfloat16*)w_down, ws.act, ws.r.topk_idx, ws.r.topk_w,
                                             ws.r.tok_class, y, d);
  }
  return cudaGetLastError();
}

template <typename XT>
__global__ void k_residual_add(XT* __restrict__ x, const float* __restrict__ y, const uint8_t* __restrict__ tok_class,
                               int T, int H) {
  const size_t n = (size_t)T * H;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    const int t = (int)(i / H);
    if (tok_class[t] == TEAM_CLS_SKIP) continue;
    const float v = to_f32(x[i]) + y[i];
    if constexpr (sizeof(XT) == 2) x[i] = __float2bfloat16_rn(v);
    else x[i] = v;
  }
}

cudaError_t launch_residual_add(void* x, int dtype, const float* y, const uint8_t* tok_class, int T, int H,
                                cudaStream_t s) {
  const size_t n = (size_t)T * H;
  const int grid = (int)((n + 255) / 256 < 1184 ? (n + 255) / 256 : 1184);
  if (dtype == TEAM_DTYPE_F32) k_residual_add<float><<<grid, 256, 0, s>>>((float*)x, y, tok_class, T, H);
  else k_residual_add<__nv_bfloat16><<<grid, 256, 0, s>>>((__nv_bfloat16*)x, y, tok_class, T, H);
  return cudaGetLastError();
}

}  // namespace team
