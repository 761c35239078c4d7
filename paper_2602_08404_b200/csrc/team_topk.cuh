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

constexpr uint32_t kKeyNegInf = 0x007fffffu;            // float_key(-inf): "not a candidate"

// Sorts a lane's eight (key, slot) pairs: key descending, equal keys by ascending slot (slot i stands for expert
// i*32+lane, so this is "ties to the lower expert id" inside the lane).  A 19-comparator network, all indices
// compile-time constants: everything stays in registers.
__device__ __forceinline__ void sort_lane_keys(uint32_t (&key)[kMaxPerLane], int (&slot)[kMaxPerLane]) {
  static_assert(kMaxPerLane == 8, "the network below sorts eight entries");
#define TEAM_CE(i, j)                                                                        \
  {                                                                                          \
    const bool sw = key[j] > key[i] || (key[j] == key[i] && slot[j] < slot[i]);              \
    const uint32_t ka = sw ? key[j] : key[i], kb = sw ? key[i] : key[j];                     \
    const int sa = sw ? slot[j] : slot[i], sb = sw ? slot[i] : slot[j];                      \
    key[i] = ka; key[j] = kb; slot[i] = sa; slot[j] = sb;                                    \
  }
  TEAM_CE(0, 1) TEAM_CE(2, 3) TEAM_CE(4, 5) TEAM_CE(6, 7)
  TEAM_CE(0, 2) TEAM_CE(1, 3) TEAM_CE(4, 6) TEAM_CE(5, 7)
  TEAM_CE(1, 2) TEAM_CE(5, 6) TEAM_CE(0, 4) TEAM_CE(3, 7)
  TEAM_CE(1, 5) TEAM_CE(2, 6)
  TEAM_CE(1, 4) TEAM_CE(3, 6)
  TEAM_CE(2, 4) TEAM_CE(3, 5)
  TEAM_CE(3, 4)
#undef TEAM_CE
}

// Core of the selection.  key[] / slot[] are the lane's candidates as sort_lane_keys leaves them (non-candidates
// carry kKeyNegInf and sort to the end).  Picks the k largest keys of the warp in descending order, ties to the
// lower expert id, and calls on_pick(j, expert, key) for the j-th pick ON THE LANE THAT HOLDS IT (nothing is
// broadcast).  Picked entries are shifted out.  Returns the number of picks made (< k only if fewer than k
// candidates exist); margin_out (all lanes) = logit of the last pick minus the best logit left (+inf if none).
//
// One pick is a short dependent chain: the warp-wide maximum of the lanes' heads (one redux), a ballot of who
// holds it, and the holder shifts its list by one; two or more holders (equal logits in different lanes) take a
// second redux for the lowest expert id.
template <typename OnPick>
__device__ __forceinline__ int warp_topk_picks(uint32_t (&key)[kMaxPerLane], int (&slot)[kMaxPerLane], int k, int lane,
                                               OnPick&& on_pick, float& margin_out) {
  float last = kNegInf;
  margin_out = __builtin_huge_valf();
  int n = 0;
  for (int j = 0; j <= k; ++j) {
    const uint32_t bk = key[0];
    const uint32_t wk = __reduce_max_sync(0xffffffffu, bk);
    if (wk == kKeyNegInf) break;                        // no candidate left
    if (j == k) {
      margin_out = last - key_float(wk);
      break;
    }
    const uint32_t holders = __ballot_sync(0xffffffffu, bk == wk);
    int win_lane = __ffs(holders) - 1;
    if (holders & (holders - 1u)) {
      const uint32_t wi = __reduce_min_sync(0xffffffffu, bk == wk ? (uint32_t)(slot[0] * 32 + lane) : 0x7fffffffu);
      win_lane = (int)(wi & 31u);
    }
    if (lane == win_lane) {
      on_pick(j, slot[0] * 32 + lane, wk);
#pragma unroll
      for (int i = 0; i + 1 < kMaxPerLane; ++i) {
        key[i] = key[i + 1];
        slot[i] = slot[i + 1];
      }
      key[kMaxPerLane - 1] = kKeyNegInf;
    }
    last = key_float(wk);
    n = j + 1;
  }
  return n;
}

// v[i] is the logit of expert i*32+lane, or -inf if that expert is not a candidate
// (beyond E, or outside the allowed set); only the first ne = ceil(E / 32) entries are looked at.
// Lane j < k receives the j-th choice.
__device__ __forceinline__ TopkResult warp_topk(const float (&v)[kMaxPerLane], int k, int lane, int ne = kMaxPerLane) {
  TopkResult r;
  r.idx = -1;
  r.val = kNegInf;
  r.top = kNegInf;
  uint32_t key[kMaxPerLane];
  int slot[kMaxPerLane];
#pragma unroll
  for (int i = 0; i < kMaxPerLane; ++i) {
    key[i] = i < ne ? float_key(v[i]) : kKeyNegInf;
    slot[i] = i;
  }
  sort_lane_keys(key, slot);
  // the holder of a pick remembers it; afterwards pick j moves to lane j (one shuffle per pick, off the picks'
  // dependent chain)
  int order[kMaxPerLane];             // this lane's key i was picked as pick number order[i] (-1: not picked)
#pragma unroll
  for (int i = 0; i < kMaxPerLane; ++i) order[i] = -1;
  const int n = warp_topk_picks(key, slot, k, lane,
                                [&](int j, int e, uint32_t) {
#pragma unroll
                                  for (int i = 0; i < kMaxPerLane; ++i)
                                    if (i == (e >> 5)) order[i] = j;
                                },
                                r.margin);
  for (int j = 0; j < n; ++j) {
    int slot = -1;
    float mine_val = 0.f;
#pragma unroll
    for (int i = 0; i < kMaxPerLane; ++i)
      if (order[i] == j) {
        slot = i;
        mine_val = v[i];
      }
    const uint32_t holder = __ballot_sync(0xffffffffu, slot >= 0);
    const int src = __ffs(holder) - 1;
    const int e = __shfl_sync(0xffffffffu, slot * 32 + lane, src);
    const float val = __shfl_sync(0xffffffffu, mine_val, src);
    if (lane == j) {
      r.idx = e;
      r.val = val;
    }
    if (j == 0) r.top = val;
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
