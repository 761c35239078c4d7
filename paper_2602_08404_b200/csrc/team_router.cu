// Router kernels (Algorithm 1 "Router"; Sec. 4.1 for which rows are computed).
//
//  k_router_logits : logits[t,e] = sum_h x[t,h] * W_r[e,h] in fp32.  The work is split over
//                    experts (one warp per expert, 128-bit loads of the expert's row) and over
//                    tiles of 8 rows whose activations sit in shared memory, so that with a
//                    handful of rows the 4*E*H bytes of router weights are still pulled by many SMs.
//                    The same launch zeroes the output rows the expert kernel will accumulate into.
//  k_router_topk   : one warp per row: softmax over all experts, plain top-k by warp shuffles,
//                    renormalised weights, decision margin (team_route's outputs).
#include <mutex>

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
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the selection kernel may stage its inputs meanwhile
  const int t0 = blockIdx.y * kRowTile;
  const int nt = min(kRowTile, d.T - t0);
  const int tid = threadIdx.x;
  const int H = d.H;
  // this warp's expert: the first batch of its weight row is requested before anything else
  const int warp = tid >> 5, lane = tid & 31;
  const int e = blockIdx.x * kExpertsPerCta + warp;
  const float4* wrow = reinterpret_cast<const float4*>(w_router + (size_t)min(e, d.E - 1) * H);
  const int n4 = H >> 2;
  constexpr int kBatch = 8;             // float4 per lane and batch: 4 KB of the row per warp in flight
  float4 wv[kBatch];
#pragma unroll
  for (int i = 0; i < kBatch; ++i)
    wv[i] = lane + 32 * i < n4 ? __ldg(wrow + lane + 32 * i) : make_float4(0.f, 0.f, 0.f, 0.f);

  if constexpr (sizeof(XT) == 2) {
    const uint2* src = reinterpret_cast<const uint2*>(x + (size_t)t0 * H);
    for (int i = tid; i < nt * H / 4; i += blockDim.x) {
      const uint2 v = __ldg(src + i);
      const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v.x));
      const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v.y));
      reinterpret_cast<float4*>(s_x)[i] = make_float4(a.x, a.y, b.x, b.y);
    }
  } else {
    const float4* src = reinterpret_cast<const float4*>(x + (size_t)t0 * H);
    for (int i = tid; i < nt * H / 4; i += blockDim.x) reinterpret_cast<float4*>(s_x)[i] = __ldg(src + i);
  }
  for (int i = nt * H + tid; i < kRowTile * H; i += blockDim.x) s_x[i] = 0.f;

  // Output rows of computed tokens start from zero (the expert kernel adds partial sums into them);
  // the CTAs of one row tile share the job.
  if (y_zero != nullptr) {
    for (int r = 0; r < nt; ++r) {
      const bool skip = (flags & TEAM_F_DCD) && tok_state[t0 + r] == TEAM_TOK_CACHED;
      if (!skip)
        for (int i = blockIdx.x * blockDim.x + tid; i < H; i += gridDim.x * blockDim.x)
          y_zero[(size_t)(t0 + r) * H + i] = 0.f;
    }
  }
  __syncthreads();

  if (e >= d.E) return;
  float acc[kRowTile];
#pragma unroll
  for (int r = 0; r < kRowTile; ++r) acc[r] = 0.f;
  // batches of kBatch float4 per lane; the next batch is requested before the current one is used
  // (the summation order over c is unchanged: ascending c within a lane)
  for (int base = 0; base < n4; base += 32 * kBatch) {
    float4 wn[kBatch];
    const int nbase = base + 32 * kBatch;
#pragma unroll
    for (int i = 0; i < kBatch; ++i)
      wn[i] = nbase + lane + 32 * i < n4 ? __ldg(wrow + nbase + lane + 32 * i) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int i = 0; i < kBatch; ++i) {
      const int c = base + lane + 32 * i;
      if (c < n4) {
        const float4 w = wv[i];
#pragma unroll
        for (int r = 0; r < kRowTile; ++r) {
          const float4 xv = *reinterpret_cast<const float4*>(s_x + r * H + c * 4);
          acc[r] = fmaf(w.x, xv.x, acc[r]);
          acc[r] = fmaf(w.y, xv.y, acc[r]);
          acc[r] = fmaf(w.z, xv.z, acc[r]);
          acc[r] = fmaf(w.w, xv.w, acc[r]);
        }
      }
    }
#pragma unroll
    for (int i = 0; i < kBatch; ++i) wv[i] = wn[i];
  }
#pragma unroll
  for (int r = 0; r < kRowTile; ++r) {
    const float s = warp_sum(acc[r]);
    if (lane == 0 && r < nt) logits[(size_t)(t0 + r) * d.E + e] = s;
  }
}


// Many rows (bf16 activations): a register-tiled fp32 FMA kernel.  A CTA takes 16 rows x 32 experts; the rows sit in
// shared memory as bf16 (widened exactly on use); warp w takes experts 4w .. 4w+3 of the tile, its lanes stride
// the hidden dimension four elements at a time (128-bit weight loads, 512 contiguous bytes per warp and expert)
// and keep 4 x 16 accumulators each, so that one weight load feeds 16 rows and one row load feeds 4 experts.  The
// 64 per-lane partial sums of a warp are reduced with a transposing butterfly (62 shuffles instead of 320).
constexpr int kTiledRows = 16;
constexpr int kTiledExperts = 32;      // per CTA: 8 warps x 4

__device__ __forceinline__ void butterfly32(float (&v)[32], int lane) {
  // after the five steps lane l holds the warp-wide sum of entry l
#pragma unroll
  for (int half = 16; half >= 1; half >>= 1) {
    const bool upper = (lane & half) != 0;
#pragma unroll
    for (int i = 0; i < half; ++i) {
      const float keep = upper ? v[i + half] : v[i];
      const float send = upper ? v[i] : v[i + half];
      v[i] = keep + __shfl_xor_sync(0xffffffffu, send, half);
    }
  }
}

__global__ void __launch_bounds__(256)
k_router_logits_tiled(const __nv_bfloat16* __restrict__ x, const float* __restrict__ w_router,
                      const uint8_t* __restrict__ tok_state, float* __restrict__ logits, float* __restrict__ y_zero,
                      Dims d, int flags) {
  extern __shared__ __align__(16) unsigned char s_xb[];   // [kTiledRows][H] bf16
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int H = d.H, T = d.T, E = d.E;
  const int t0 = blockIdx.y * kTiledRows, nt = min(kTiledRows, T - t0);
  const int e0 = blockIdx.x * kTiledExperts + warp * 4;
  // stage the rows (16-byte pieces; rows beyond T are zero)
  {
    const uint4* src = reinterpret_cast<const uint4*>(x + (size_t)t0 * H);
    uint4* dst = reinterpret_cast<uint4*>(s_xb);
    const int n16 = nt * H / 8, all16 = kTiledRows * H / 8;
    for (int i = tid; i < all16; i += 256) dst[i] = i < n16 ? __ldg(src + i) : make_uint4(0u, 0u, 0u, 0u);
  }
  if (y_zero != nullptr) {
    for (int r = 0; r < nt; ++r) {
      const bool skip = (flags & TEAM_F_DCD) && tok_state[t0 + r] == TEAM_TOK_CACHED;
      if (!skip)
        for (int i = blockIdx.x * 256 + tid; i < H; i += gridDim.x * 256) y_zero[(size_t)(t0 + r) * H + i] = 0.f;
    }
  }
  __syncthreads();
  float acc[2][32];                    // [pair of experts][expert-in-pair * 16 + row]
#pragma unroll
  for (int g = 0; g < 2; ++g)
#pragma unroll
    for (int i = 0; i < 32; ++i) acc[g][i] = 0.f;
  const float4* wrow[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) wrow[q] = reinterpret_cast<const float4*>(w_router + (size_t)min(e0 + q, E - 1) * H);
  const int n4 = H >> 2;
  float4 wv[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) wv[q] = __ldg(wrow[q] + lane);
  for (int c = lane; c < n4; c += 32) {
    float4 wn[4];
    const int cn = c + 32 < n4 ? c + 32 : c;             // next step's weights are requested before this step's math
#pragma unroll
    for (int q = 0; q < 4; ++q) wn[q] = __ldg(wrow[q] + cn);
#pragma unroll
    for (int r = 0; r < kTiledRows; ++r) {
      const uint2 xb = *reinterpret_cast<const uint2*>(s_xb + ((size_t)r * H + c * 4) * 2);
      const float2 lo = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&xb.x));
      const float2 hi = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&xb.y));
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        float a = acc[q >> 1][(q & 1) * 16 + r];
        a = fmaf(wv[q].x, lo.x, a);
        a = fmaf(wv[q].y, lo.y, a);
        a = fmaf(wv[q].z, hi.x, a);
        a = fmaf(wv[q].w, hi.y, a);
        acc[q >> 1][(q & 1) * 16 + r] = a;
      }
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) wv[q] = wn[q];
  }
#pragma unroll
  for (int g = 0; g < 2; ++g) {
    butterfly32(acc[g], lane);
    const int e = e0 + g * 2 + (lane >> 4), r = lane & 15;
    if (e < E && r < nt) logits[(size_t)(t0 + r) * E + e] = acc[g][0];
  }
}

// Few rows (T <= kRowTile): the whole job is one pass over the 4*E*H bytes of router weights, so it
// is spread as widely as possible -- two experts per CTA, four warps per expert, each lane issuing all
// of its 128-bit weight loads before anything else -- and the activations are staged once per CTA.
constexpr int kSmallExperts = 2;   // experts per CTA
constexpr int kSmallSplit = 4;     // warps per expert (each takes H/4 of the dot product)
constexpr int kSmallMaxVec = 8;    // float4 per lane: supports H <= 4096

template <typename XT>
__global__ void __launch_bounds__(kSmallExperts * kSmallSplit * 32)
k_router_logits_small(const XT* __restrict__ x, const float* __restrict__ w_router,
                      const uint8_t* __restrict__ tok_state, float* __restrict__ logits, float* __restrict__ y_zero,
                      Dims d, int flags) {
  extern __shared__ __align__(16) float s_x[];   // [T][H] then partial sums
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the selection kernel may stage its inputs meanwhile
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int H = d.H, T = d.T;
  const int e = blockIdx.x * kSmallExperts + warp / kSmallSplit;
  const int part = warp % kSmallSplit;
  const int n4 = H >> 2, per_part = n4 / kSmallSplit;   // float4 per warp

  // 1. weights first: every load in flight at once
  float4 w[kSmallMaxVec];
  const float4* wrow = reinterpret_cast<const float4*>(w_router + (size_t)min(e, d.E - 1) * H) + part * per_part;
#pragma unroll
  for (int i = 0; i < kSmallMaxVec; ++i)
    w[i] = (lane + 32 * i < per_part) ? __ldg(wrow + lane + 32 * i) : make_float4(0.f, 0.f, 0.f, 0.f);

  // 2. stage the rows (16-byte loads), zero this CTA's share of the output rows
  if constexpr (sizeof(XT) == 2) {
    const uint4* src = reinterpret_cast<const uint4*>(x);
    for (int i = tid; i < T * H / 8; i += blockDim.x) {
      const uint4 v = __ldg(src + i);
      const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&v);
      float4 lo, hi;
      float2 f;
      f = __bfloat1622float2(p[0]); lo.x = f.x; lo.y = f.y;
      f = __bfloat1622float2(p[1]); lo.z = f.x; lo.w = f.y;
      f = __bfloat1622float2(p[2]); hi.x = f.x; hi.y = f.y;
      f = __bfloat1622float2(p[3]); hi.z = f.x; hi.w = f.y;
      reinterpret_cast<float4*>(s_x)[2 * i] = lo;
      reinterpret_cast<float4*>(s_x)[2 * i + 1] = hi;
    }
  } else {
    const float4* src = reinterpret_cast<const float4*>(x);
    for (int i = tid; i < T * H / 4; i += blockDim.x) reinterpret_cast<float4*>(s_x)[i] = __ldg(src + i);
  }
  if (y_zero != nullptr) {
    const int total4 = T * H / 4;
    for (int i = blockIdx.x * blockDim.x + tid; i < total4; i += gridDim.x * blockDim.x) {
      const int t = (i * 4) / H;
      const bool skip = (flags & TEAM_F_DCD) && tok_state[t] == TEAM_TOK_CACHED;
      if (!skip) reinterpret_cast<float4*>(y_zero)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
  }
  __syncthreads();

  // 3. partial dot products, warp reduction, then the four parts of each expert are added in a fixed order
  float acc[kRowTile];
#pragma unroll
  for (int r = 0; r < kRowTile; ++r) acc[r] = 0.f;
#pragma unroll
  for (int i = 0; i < kSmallMaxVec; ++i) {
    if (lane + 32 * i < per_part) {
      const int c = part * per_part + lane + 32 * i;
#pragma unroll
      for (int r = 0; r < kRowTile; ++r) {
        if (r < T) {
          const float4 xv = *reinterpret_cast<const float4*>(s_x + r * H + c * 4);
          acc[r] = fmaf(w[i].x, xv.x, acc[r]);
          acc[r] = fmaf(w[i].y, xv.y, acc[r]);
          acc[r] = fmaf(w[i].z, xv.z, acc[r]);
          acc[r] = fmaf(w[i].w, xv.w, acc[r]);
        }
      }
    }
  }
  float* s_part = s_x + T * H;   // [warps][kRowTile]
#pragma unroll
  for (int r = 0; r < kRowTile; ++r) {
    const float sum = warp_sum(acc[r]);
    if (lane == 0) s_part[warp * kRowTile + r] = sum;
  }
  __syncthreads();
  if (tid < kSmallExperts * kRowTile) {
    const int le = tid / kRowTile, r = tid % kRowTile;
    const int ee = blockIdx.x * kSmallExperts + le;
    if (ee < d.E && r < T) {
      float sum = 0.f;
#pragma unroll
      for (int q = 0; q < kSmallSplit; ++q) sum += s_part[(le * kSmallSplit + q) * kRowTile + r];
      logits[(size_t)r * d.E + ee] = sum;
    }
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
  TopkResult r = warp_topk(v, d.k, lane, (d.E + 31) / 32);
  const float w = routing_weight(r, d.k, lane, row_max, denom, p.norm_topk);
  if (lane < d.k) {
    if (out.topk_idx) out.topk_idx[t * d.k + lane] = r.idx;
    if (out.topk_w) out.topk_w[t * d.k + lane] = w;
  }
  if (lane == 0 && out.margin) out.margin[t] = r.margin;
}

// Opt in to the dynamic shared memory the kernels need (done once per context, outside any stream capture).
static bool small_router_ok(const Dims& d) {
  return d.T <= kRowTile && d.H % (4 * kSmallSplit) == 0 && d.H / (4 * kSmallSplit) <= 32 * kSmallMaxVec;
}

// All kernels of the layer ask for the largest shared-memory carve-out, as the expert kernel must:
// an SM whose carve-out differs from what the next kernel prefers is drained and reconfigured first.
template <typename K>
static cudaError_t prepare_kernel(K kernel, int smem) {
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
  return e;
}

// The opt-in is a per-device property of the kernel, shared by every context (and by the context-free
// entry point): it is only ever raised, so that preparing for a small hidden size cannot take away
// what a larger one needs.
int router_smem_bytes(int hidden) { return kRowTile * hidden * (int)sizeof(float) + 1024; }

cudaError_t configure_router(int dtype, int hidden) {
  static std::mutex mu;
  static int prepared[64][2] = {};   // [device][dtype]: shared-memory bytes opted in so far
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const int smem = router_smem_bytes(hidden);
  const int di = dtype == TEAM_DTYPE_F32 ? 0 : 1;
  std::lock_guard<std::mutex> lock(mu);
  if (dev >= 0 && dev < 64 && prepared[dev][di] >= smem) return cudaSuccess;
  if (dtype == TEAM_DTYPE_F32) {
    e = prepare_kernel(k_router_logits<float>, smem);
    if (e == cudaSuccess) e = prepare_kernel(k_router_logits_small<float>, smem);
  } else {
    e = prepare_kernel(k_router_logits<__nv_bfloat16>, smem);
    if (e == cudaSuccess) e = prepare_kernel(k_router_logits_small<__nv_bfloat16>, smem);
    if (e == cudaSuccess) e = prepare_kernel(k_router_logits_tiled, smem);
  }
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(k_router_topk, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
  if (e == cudaSuccess && dev >= 0 && dev < 64) prepared[dev][di] = smem;
  return e;
}

cudaError_t launch_router_logits(const void* x, int dtype, const float* w_router, const uint8_t* tok_state,
                                 float* logits, float* y_zero, Dims d, int flags, cudaStream_t s) {
  if (small_router_ok(d)) {
    dim3 grid((d.E + kSmallExperts - 1) / kSmallExperts), block(kSmallExperts * kSmallSplit * 32);
    const size_t smem = (size_t)d.T * d.H * sizeof(float) + kSmallExperts * kSmallSplit * kRowTile * sizeof(float);
    if (dtype == TEAM_DTYPE_F32)
      k_router_logits_small<float><<<grid, block, smem, s>>>(static_cast<const float*>(x), w_router, tok_state,
                                                             logits, y_zero, d, flags);
    else
      k_router_logits_small<__nv_bfloat16><<<grid, block, smem, s>>>(static_cast<const __nv_bfloat16*>(x), w_router,
                                                                     tok_state, logits, y_zero, d, flags);
    return cudaGetLastError();
  }
  // the register-tiled kernel pays off once its 16-row x 32-expert tiles fill the SMs; smaller calls keep more,
  // smaller CTAs in flight with the 8 x 8 kernel below
  if (dtype == TEAM_DTYPE_BF16 && ((d.T + kTiledRows - 1) / kTiledRows) * ((d.E + kTiledExperts - 1) / kTiledExperts) >= 128) {
    dim3 grid((d.E + kTiledExperts - 1) / kTiledExperts, (d.T + kTiledRows - 1) / kTiledRows);
    k_router_logits_tiled<<<grid, 256, (size_t)kTiledRows * d.H * 2, s>>>(static_cast<const __nv_bfloat16*>(x), w_router,
                                                                        tok_state, logits, y_zero, d, flags);
    return cudaGetLastError();
  }
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
