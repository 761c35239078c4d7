// Shared by the two attention kernels (Sec. 4.1, the attention half of delayed caching): argument block and
// the test for "this row is computed".
#pragma once

#include "team_common.cuh"

namespace team {

constexpr int kAttnPairs = 128;        // (row, head) pairs per CTA
constexpr int kAttnMaxSplits = 8;      // portable cluster size

struct AttnArgs {
  const __nv_bfloat16* q;        // [T, Hq, d]
  const __nv_bfloat16* k_new;    // [T, Hkv, d]
  const __nv_bfloat16* v_new;
  const __nv_bfloat16* k_prefix; // [S, P, Hkv, d]
  const __nv_bfloat16* v_prefix;
  const int32_t* prefix_len;     // [S]
  __nv_bfloat16* k_block;        // [S, L, Hkv, d]
  __nv_bfloat16* v_block;
  const uint8_t* tok_state;      // [T]
  const int32_t* pos;
  const int32_t* group;
  const int32_t* branch;
  float* out;                    // [T, Hq, d]
  int32_t* status;               // [2] optional
  int S, B, L, Hq, Hkv, d, P, flags;
};

__device__ __forceinline__ bool attn_computed(int state, int flags) { return !((flags & TEAM_F_DCD) && state == TEAM_TOK_CACHED); }

// head size 128 on the tensor-memory path (team_attn_tc.cu): launch and one-time set-up
cudaError_t configure_attention_tc();
cudaError_t launch_attention_tc(const AttnArgs& a, int m_tiles, int n_splits, cudaStream_t s);

}  // namespace team
