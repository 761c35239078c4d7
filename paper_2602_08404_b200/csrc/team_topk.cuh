// Warp-level top-k over one row of router logits (Algorithm 1 "Router" / "top-k").
// One warp owns one row; lane l holds the logits of experts l, l+32, l+64, ...
// Selection is by logit, descending, ties to the lower expert id, and is exact
// (no floating-point arithmetic takes part in the decision).
#pragma once

#include "team_common.cuh"

namespace team {

constexpr int kMaxPerLane = TEAM_MAX_EXPERTS / 32;   // 8
constexpr float kNegInf = -__builtin_huge_valf();

struct TopkResult {
  int idx;        // lane j < k: id of the j-th choice (others: -1)
  float val;      // lane j < k: its logit
  float margin;   // all lanes: logit[k-1] - best logit left out (+inf if none left)
  float top;      // all lanes: largest candidate logit
};

// v[i] is the logit of expert i*32+lane, or -inf if that expert is not a candidate
// (beyond E, or outside the allowed set).  v is consumed.
__device__ __forceinline__ TopkResult warp_topk(float (&v)[kMaxPerLane], int k, int lane) {
  TopkResult r;
  r.idx = -1;
  r.val = kNegInf;
  r.top = kNegInf;
  float last = kNegInf;
  for (int j = 0; j <= k; ++j) {
    float bv = kNegInf;
    int bi = 0x7fffffff;
#pragma unroll
    for (int i = 0; i < kMaxPerLane; ++i) {
      // ascending expert id within the lane, strict '>' keeps the lower id on ties
      if (v[i] > bv) {
        bv = v[i];
        bi = i * 32 + lane;
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (ov > bv || (ov == bv && oi < bi)) {
        bv = ov;
        bi = oi;
      }
    }
    if (j == 0) r.top = bv;
    if (j < k) {
      if (lane == j) {
        r.idx = (bv == kNegInf) ? -1 : bi;
        r.val = bv;
      }
      last = bv;
      if (bv != kNegInf && (bi & 31) == lane) {
#pragma unroll
        for (int i = 0; i < kMaxPerLane; ++i)
          if (i == (bi >> 5)) v[i] = kNegInf;
      }
    } else {
      r.margin = (bv == kNegInf) ? __builtin_huge_valf() : last - bv;
    }
  }
  return r;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Loads one logits row into lane-strided registers and returns the row maximum
// and sum of exp(l - max) over all E experts (the softmax denominator).
__device__ __forceinline__ void load_row(const float* __restrict__ row, int E, int lane, float (&v)[kMaxPerLane],
                                         float& row_max, float& denom) {
  float m = kNegInf;
#pragma unroll
  for (int i = 0; i < kMaxPerLane; ++i) {
    int e = i * 32 + lane;
    v[i] = (e < E) ? row[e] : kNegInf;
    m = fmaxf(m, v[i]);
  }
  row_max = warp_max(m);
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < kMaxPerLane; ++i)
    if (i * 32 + lane < E) s += expf(v[i] - row_max);
  denom = warp_sum(s);
}

// Routing weight of lane j's choice: softmax probability, renormalised over the k chosen if asked.
__device__ __forceinline__ float routing_weight(const TopkResult& r, int k, int lane, float row_max, float denom,
                                                int norm_topk) {
  float p = (lane < k && r.idx >= 0) ? expf(r.val - row_max) : 0.f;
  float s = norm_topk ? warp_sum(p) : denom;
  return p / s;
}

}  // namespace team
