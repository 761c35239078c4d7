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

// Order-preserving map from a float to an unsigned key (larger float <-> larger key; -inf maps below
// every finite value), so that the warp-wide maximum is one redux instruction.
__device__ __forceinline__ uint32_t float_key(float f) {
  const uint32_t u = __float_as_uint(f + 0.0f);   // -0 and +0 compare equal: both take +0's key
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_float(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// v[i] is the logit of expert i*32+lane, or -inf if that expert is not a candidate
// (beyond E, or outside the allowed set); only the first ne = ceil(E / 32) entries are looked at.
// The logits are turned into keys once.  Each of the k+1 rounds takes the warp-wide maximum key and
// then the lowest expert id among the lanes that hold it, and retires that key.
__device__ __forceinline__ TopkResult warp_topk(const float (&v)[kMaxPerLane], int k, int lane, int ne = kMaxPerLane) {
  TopkResult r;
  r.idx = -1;
  r.val = kNegInf;
  r.top = kNegInf;
  r.margin = __builtin_huge_valf();
  float last = kNegInf;
  const uint32_t key_neg_inf = float_key(kNegInf);
  uint32_t key[kMaxPerLane];
#pragma unroll
  for (int i = 0; i < kMaxPerLane; ++i) key[i] = i < ne ? float_key(v[i]) : key_neg_inf;
  for (int j = 0; j <= k; ++j) {
    uint32_t bk = key_neg_inf;
    int bi = 0;
#pragma unroll
    for (int i = 0; i < kMaxPerLane; ++i) {
      if (i >= ne) break;
      // ascending expert id within the lane, strict '>' keeps the lower id on ties
      if (key[i] > bk) {
        bk = key[i];
        bi = i;
      }
    }
    const uint32_t wk = __reduce_max_sync(0xffffffffu, bk);
    const bool none = wk == key_neg_inf;
    const int wi = (int)__reduce_min_sync(0xffffffffu, (bk == wk && !none) ? (uint32_t)(bi * 32 + lane) : 0x7fffffffu);
    const float bv = none ? kNegInf : key_float(wk);
    if (j == 0) r.top = bv;
    if (j < k) {
      if (lane == j) {
        r.idx = none ? -1 : wi;
        r.val = bv;
      }
      last = bv;
      if (!none && (wi & 31) == lane) {
#pragma unroll
        for (int i = 0; i < kMaxPerLane; ++i)
          if (i == (wi >> 5)) key[i] = key_neg_inf;
      }
    } else {
      r.margin = none ? __builtin_huge_valf() : last - bv;
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
