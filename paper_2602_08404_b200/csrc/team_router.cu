// Router kernels (Algorithm 1 "Router"; Sec. 4.1 for which rows are computed).
//
//  k_router_logits : logits[t,e] = sum_h x[t,h] * W_r[e,h] in fp32.  The work is split over
//                    experts (one warp per expert, 128-bit loads of the expert's row) and over
//                    tiles of 8 rows whose activations sit in shared memory, so that with a
//                    handful of rows the 4*E*H bytes of router weights are still pulled by many SMs.
//                    The same launch zeroes the output rows the expert kernel will accumulate into.
//  k_router_topk   : one warp per row: softmax over all experts, plain top-k by warp shuffles,
//                    renormalised weights, decision margin (team_route's outputs).
#include "team_common.cuh"
#include "team_topk.cuh"

namespace team {

constexpr int kRowTile = 8;       // rows per CTA in the logits kernel
constexpr int kExpertsPerCta = 8; // one warp each

template <typename XT>
__global__ void __launch_bounds__(kExpertsPerCta * 32)
k_router_logits(const XT* __restrict__ x, const float* __restrict__ w_router, const uint8_t* __restrict__ tok_state,
                float* __restrict__ logits, float* __restrict__ y_zero, Dims d, int flags) {
  extern __shared__ __align__(16) float s_x[];   // [kRowTile][H]
  const int t0 = blockIdx.y * kRowTile;
  const int nt = min(kRowTile, d.T - t0);
  const int tid = threadIdx.x;
  const int H = d.H;

  for (int i = tid; i < nt * H; i += blockDim.x) s_x[i] = to_f32(x[(size_t)t0 * H + i]);
  for (int i = nt * H + tid; i < kRowTile * H; i += blockDim.x) s_x[i] = 0.f;

  // Output rows of computed tokens start from zero (the expert kernel adds partial sums into them).
  if (y_zero != nullptr && blockIdx.x == 0) {
    for (int r = 0; r < nt; ++r) {
      const bool skip = (flags & TEAM_F_DCD) && tok_state[t0 + r] == TEAM_TOK_CACHED;
      if (!skip)
        for (int i = tid; i < H; i += blockDim.x) y_zero[(size_t)(t0 + r) * H + i] = 0.f;
    }
  }
  __syncthreads();

  const int warp = tid >> 5, lane = tid & 31;
  const int e = blockIdx.x * kExpertsPerCta + warp;
  if (e >= d.E) return;
  const float4* wrow = reinterpret_cast<const float4*>(w_router + (size_t)e * H);
  float acc[kRowTile];
#pragma unroll
  for (int r = 0; r < kRowTile; ++r) acc[r] = 0.f;
  const int n4 = H >> 2;
#pragma unroll 4
  for (int c = lane; c < n4; c += 32) {
    const float4 w = __ldg(wrow + c);
#pragma unroll
    for (int r = 0; r < kRowTile; ++r) {
      const float4 xv = *reinterpret_cast<const float4*>(s_x + r * H + c * 4);
      acc[r] = fmaf(w.x, xv.x, acc[r]);
      acc[r] = fmaf(w.y, xv.y, acc[r]);
      acc[r] = fmaf(w.z, xv.z, acc[r]);
      acc[r] = fmaf(w.w, xv.w, acc[r]);
    }
  }
#pragma unroll
  for (int r = 0; r < kRowTile; ++r) {
    const float s = warp_sum(acc[r]);
    if (lane == 0 && r < nt) logits[(size_t)(t0 + r) * d.E + e] = s;
  }
}

__global__ void __launch_bounds__(256)
k_router_topk(const float* __restrict__ logits, const uint8_t* __restrict__ tok_state, RoutePtrs out, Dims d,
              Policy p) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (warp >= d.T) return;
  const int t = warp;
  const bool skip = (p.flags & TEAM_F_DCD) && tok_state[t] == TEAM_TOK_CACHED;
  if (skip) {
    if (out.probs)
      for (int e = lane; e < d.E; e += 32) out.probs[(size_t)t * d.E + e] = 0.f;
    if (lane < d.k) {
      if (out.topk_idx) out.topk_idx[t * d.k + lane] = -1;
      if (out.topk_w) out.topk_w[t * d.k + lane] = 0.f;
    }
    if (lane == 0 && out.margin) out.margin[t] = __builtin_huge_valf();
    return;
  }
  float v[kMaxPerLane];
  float row_max, denom;
  load_row(logits + (size_t)t * d.E, d.E, lane, v, row_max, denom);
  if (out.probs) {
#pragma unroll
    for (int i = 0; i < kMaxPerLane; ++i) {
      const int e = i * 32 + lane;
      if (e < d.E) out.probs[(size_t)t * d.E + e] = expf(v[i] - row_max) / denom;
    }
  }
  TopkResult r = warp_topk(v, d.k, lane);
  const float w = routing_weight(r, d.k, lane, row_max, denom, p.norm_topk);
  if (lane < d.k) {
    if (out.topk_idx) out.topk_idx[t * d.k + lane] = r.idx;
    if (out.topk_w) out.topk_w[t * d.k + lane] = w;
  }
  if (lane == 0 && out.margin) out.margin[t] = r.margin;
}

// Opt in to the dynamic shared memory the kernels need (done once per context, outside any stream capture).
cudaError_t configure_router(int dtype, int hidden) {
  const int smem = kRowTile * hidden * (int)sizeof(float);
  if (dtype == TEAM_DTYPE_F32)
    return cudaFuncSetAttribute(k_router_logits<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  return cudaFuncSetAttribute(k_router_logits<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
}

cudaError_t launch_router_logits(const void* x, int dtype, const float* w_router, const uint8_t* tok_state,
                                 float* logits, float* y_zero, Dims d, int flags, cudaStream_t s) {
  dim3 grid((d.E + kExpertsPerCta - 1) / kExpertsPerCta, (d.T + kRowTile - 1) / kRowTile);
  dim3 block(kExpertsPerCta * 32);
  const size_t smem = (size_t)kRowTile * d.H * sizeof(float);
  if (dtype == TEAM_DTYPE_F32) {
    k_router_logits<float><<<grid, block, smem, s>>>(static_cast<const float*>(x), w_router, tok_state, logits,
                                                     y_zero, d, flags);
  } else {
    k_router_logits<__nv_bfloat16><<<grid, block, smem, s>>>(static_cast<const __nv_bfloat16*>(x), w_router,
                                                             tok_state, logits, y_zero, d, flags);
  }
  return cudaGetLastError();
}

cudaError_t launch_router_topk(const float* logits, const uint8_t* tok_state, RoutePtrs out, Dims d, Policy p,
                               cudaStream_t s) {
  const int warps_per_block = 8;
  dim3 grid((d.T + warps_per_block - 1) / warps_per_block);
  k_router_topk<<<grid, warps_per_block * 32, 0, s>>>(logits, tok_state, out, d, p);
  return cudaGetLastError();
}

}  // namespace team
