// Decode-loop glue of one block (Eq. 2-3; Sec. 4.2 and Sec. 5.4): threshold acceptance, chained verification of
// the speculative branches, the next pair of candidates, and the rows of the next forward pass.  Integer and
// compare work only: one warp per sequence, lane = position (blocks of at most 64 positions, two per lane).
#include "team_common.cuh"
#include "team_topk.cuh"

namespace team {

struct SehArgs {
  int32_t* token;         // [S, L]   accepted token, -1 while masked
  uint8_t* state;         // [S, L]   TEAM_TOK_*
  int32_t* spec_pos;      // [S, 2]   candidates of the forward pass whose outputs are given (-1: none)
  int32_t* spec_tok;      // [S, 2]
  int32_t* counters;      // [S, 2]   forward passes, accepted tokens (accumulated); may be null
  const int32_t* pred;    // [S, B, L] predicted token per branch and position (null: begin a block)
  const float* conf;      // [S, B, L]
  uint8_t* r_state;       // rows of the next forward pass, [S, B, L] each
  float* r_conf;
  int32_t* r_pos;
  int32_t* r_group;
  int32_t* r_branch;
  int32_t* adopted;       // [S] may be null
  int S, L, B;
  float tau;
};

__global__ void __launch_bounds__(128) k_seh_step(SehArgs a) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= a.S) return;
  const int s = warp, L = a.L, B = a.B;
  const bool begin = a.pred == nullptr;
  int sp0 = -1, sp1 = -1, tk0 = -1, tk1 = -1;
  if (!begin && B == 4) {
    sp0 = a.spec_pos[s * 2];
    sp1 = a.spec_pos[s * 2 + 1];
    tk0 = a.spec_tok[s * 2];
    tk1 = a.spec_tok[s * 2 + 1];
  }
  const int32_t* pred = begin ? nullptr : a.pred + (size_t)s * B * L;
  const float* conf = begin ? nullptr : a.conf + (size_t)s * B * L;
  auto confirmed = [&](int b, int pos, int tok) {
    return pos >= 0 && pred[b * L + pos] == tok && conf[b * L + pos] > a.tau;
  };
  // ---- the chain of trusted branches (Sec. 5.4) ----
  int second = -1;                   // the branch trusted after the base one: 1, 2 or none
  bool third = false;                // ... and branch 3 after it
  if (!begin && B == 4) {
    if (confirmed(0, sp0, tk0)) {
      second = 1;
      third = confirmed(1, sp1, tk1);
    } else if (confirmed(0, sp1, tk1)) {
      second = 2;
      third = confirmed(2, sp0, tk0);
    }
  }
  const int adopted = third ? 3 : (second > 0 ? second : 0);
  // ---- acceptance (Eq. 3) along the chain, state update (Sec. 4.1) ----
  int nst[2], n_new = 0;
  float cadopt[2];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int p = lane + 32 * h;
    nst[h] = TEAM_TOK_CACHED;
    cadopt[h] = 0.f;
    if (p >= L) continue;
    if (begin) {
      a.token[s * L + p] = -1;
      a.state[s * L + p] = TEAM_TOK_MASKED;
      nst[h] = TEAM_TOK_MASKED;
      continue;
    }
    const int st = a.state[s * L + p];
    int newly = -1;
    bool got = false;
    auto visit = [&](int b) {
      const bool s0 = (b == 1 || b == 3) && sp0 == p, s1 = (b == 2 || b == 3) && sp1 == p;
      if (!got && s0) { newly = tk0; got = true; }
      if (!got && s1) { newly = tk1; got = true; }
      if (!got && st == TEAM_TOK_MASKED && !s0 && !s1 && conf[b * L + p] > a.tau) { newly = pred[b * L + p]; got = true; }
    };
    visit(0);
    if (second > 0) visit(second);
    if (third) visit(3);
    int ns = st == TEAM_TOK_NEW ? TEAM_TOK_CACHED : st;
    if (got) {
      ns = TEAM_TOK_NEW;
      a.token[s * L + p] = newly;
      ++n_new;
    }
    a.state[s * L + p] = (uint8_t)ns;
    nst[h] = ns;
    cadopt[h] = conf[adopted * L + p];
  }
  n_new = __reduce_add_sync(0xffffffffu, n_new);
  // ---- the next two candidates: highest confidences of the adopted branch among the positions still masked ----
  int c_pos[2] = {-1, -1};
  if (!begin && B == 4) {
    uint32_t key[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) key[h] = (lane + 32 * h < L && nst[h] == TEAM_TOK_MASKED) ? float_key(cadopt[h]) : 0u;
    for (int i = 0; i < 2; ++i) {
      const uint32_t mine = key[0] >= key[1] ? key[0] : key[1];
      const uint32_t best = __reduce_max_sync(0xffffffffu, mine);
      if (best == 0u) break;                                              // nothing masked is left
      // the lowest position among all holders of the best key (a lane may hold it at both of its positions)
      uint32_t cand = 0xffffu;
#pragma unroll
      for (int h = 0; h < 2; ++h)
        if (key[h] == best) cand = min(cand, (uint32_t)(lane + 32 * h));
      const uint32_t win = __reduce_min_sync(0xffffffffu, cand);
      c_pos[i] = (int)win;
#pragma unroll
      for (int h = 0; h < 2; ++h)
        if ((int)win == lane + 32 * h) key[h] = 0u;
    }
  }
  if (lane == 0) {
    if (!begin && B == 4) {
      a.spec_pos[s * 2] = c_pos[0];
      a.spec_pos[s * 2 + 1] = c_pos[1];
      a.spec_tok[s * 2] = c_pos[0] >= 0 ? pred[adopted * L + c_pos[0]] : -1;
      a.spec_tok[s * 2 + 1] = c_pos[1] >= 0 ? pred[adopted * L + c_pos[1]] : -1;
    } else {
      a.spec_pos[s * 2] = a.spec_pos[s * 2 + 1] = -1;
      a.spec_tok[s * 2] = a.spec_tok[s * 2 + 1] = -1;
    }
    if (a.adopted) a.adopted[s] = adopted;
    if (a.counters) {
      if (begin) {
        a.counters[s * 2] = a.counters[s * 2 + 1] = 0;
      } else {
        a.counters[s * 2] += 1;
        a.counters[s * 2 + 1] += n_new;
      }
    }
  }
  // ---- rows of the next forward pass: [branch][position] ----
  for (int b = 0; b < B; ++b) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int p = lane + 32 * h;
      if (p >= L) continue;
      int st = nst[h];
      if ((b == 1 || b == 3) && p == c_pos[0]) st = TEAM_TOK_NEW;
      if ((b == 2 || b == 3) && p == c_pos[1]) st = TEAM_TOK_NEW;
      const size_t r = ((size_t)s * B + b) * L + p;
      a.r_state[r] = (uint8_t)st;
      a.r_conf[r] = st == TEAM_TOK_MASKED ? cadopt[h] : 1.f;
      a.r_pos[r] = p;
      a.r_group[r] = s;
      a.r_branch[r] = b;
    }
  }
}

}  // namespace team

extern "C" int team_seh_step(const team_seh_config* cfg, const team_seh_state* state, const int32_t* pred, const float* conf,
                             const team_seh_rows* rows, int32_t* adopted_out, void* stream) {
  if (cfg == nullptr || state == nullptr || rows == nullptr) return TEAM_ERR_ARG;
  if (cfg->n_seqs < 1 || cfg->block < 1 || cfg->block > TEAM_MAX_BLOCK) return TEAM_ERR_SHAPE;
  if (cfg->n_branches != 1 && cfg->n_branches != 4) return TEAM_ERR_SHAPE;
  if ((long long)cfg->n_seqs * cfg->n_branches * cfg->block > TEAM_MAX_ROWS) return TEAM_ERR_SHAPE;
  if (!state->token || !state->state || !state->spec_pos || !state->spec_tok) return TEAM_ERR_ARG;
  if (!rows->tok_state || !rows->conf || !rows->pos || !rows->group || !rows->branch) return TEAM_ERR_ARG;
  if ((pred == nullptr) != (conf == nullptr)) return TEAM_ERR_ARG;
  team::SehArgs a;
  a.token = state->token; a.state = state->state; a.spec_pos = state->spec_pos; a.spec_tok = state->spec_tok;
  a.counters = state->counters;
  a.pred = pred; a.conf = conf;
  a.r_state = rows->tok_state; a.r_conf = rows->conf; a.r_pos = rows->pos; a.r_group = rows->group; a.r_branch = rows->branch;
  a.adopted = adopted_out;
  a.S = cfg->n_seqs; a.L = cfg->block; a.B = cfg->n_branches; a.tau = cfg->tau;
  const int warps_per_block = 4;
  team::k_seh_step<<<(cfg->n_seqs + warps_per_block - 1) / warps_per_block, warps_per_block * 32, 0,
                     static_cast<cudaStream_t>(stream)>>>(a);
  return cudaGetLastError() == cudaSuccess ? TEAM_OK : TEAM_ERR_CUDA;
}
