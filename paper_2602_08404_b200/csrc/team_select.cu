// Selection / permutation kernel: Eq. 4 classification, Algorithm 1's two routing rounds, the
// necessary expert set E_A per group, and the dispatch tables (per-expert counts, exclusive
// offsets, the expert-sorted slot permutation, the active-expert list and the expert kernel's
// work items).  One CTA of 1024 threads; all cross-row state (group masks, histograms, scans)
// lives in shared memory.
//
// Layout contract: rows with equal (group, branch) are contiguous (one decoding block, at most
// TEAM_MAX_BLOCK rows), so the "distance to a decoded token" test of Eq. 4 only walks a row's own run.
#include <cooperative_groups.h>

#include <mutex>

#include "team_common.cuh"
#include "team_topk.cuh"

namespace team {

namespace cg = cooperative_groups;

constexpr int kSelThreads = 1024;
constexpr int kSelWarps = kSelThreads / 32;

constexpr int kIdxInSmemMax = 8192;   // routed slots kept in shared memory between the rounds and the dispatch
enum { kSelAll = 0, kSelRounds = 1, kSelDispatch = 2, kSelCluster = 3 };   // what one launch of the kernel does
constexpr int kSmallSlots = 128;      // up to here every expert's thread counts and places its slots by itself

struct SelSmem {
  // carved from dynamic shared memory in this order
  uint32_t* mask;      // [G][8]  E_A bits (256 experts max)
  uint32_t* mask2;     // [G][8]  cluster mode: the union over the cluster's CTAs while it is being formed
  int32_t* hist;       // [kSelWarps][E+ns]
  int32_t* off;        // [E+ns+1]
  int32_t* key;        // [T] group*256 + branch
  int32_t* pos;        // [T]
  int32_t* warp_cnt;   // [kSelWarps + 1]
  int32_t* scan_tot;   // [3][kSelWarps] per-warp totals of the scan over experts: slots, work items, active experts
  int32_t* idx;        // [min(T*k, kIdxInSmemMax)]
  uint8_t* state;      // [T]
  uint8_t* cls;        // [T]
  uint8_t* has_first;  // [G]
  int32_t* own;        // [T + 1] kSelRounds: the rows this CTA routes, own[T] = how many
};

__host__ __device__ inline size_t sel_smem_layout(Dims d, SelSmem* s, unsigned char* base) {
  size_t o = 0;
  auto take = [&](size_t bytes) {
    size_t at = o;
    o += (bytes + 15) & ~size_t(15);
    return at;
  };
  const int EN = d.E + d.ns;
  const int n_idx = d.T * d.k <= kIdxInSmemMax ? d.T * d.k : 0;
  size_t a_mask = take((size_t)d.G * 8 * 4);
  size_t a_mask2 = take((size_t)d.G * 8 * 4);
  size_t a_hist = take((size_t)kSelWarps * EN * 4);
  size_t a_off = take((size_t)(EN + 1) * 4);
  size_t a_key = take((size_t)d.T * 4);
  size_t a_pos = take((size_t)d.T * 4);
  size_t a_wc = take((size_t)(kSelWarps + 1) * 4);
  size_t a_st = take((size_t)3 * kSelWarps * 4);
  size_t a_idx = take((size_t)n_idx * 4);
  size_t a_state = take((size_t)d.T);
  size_t a_cls = take((size_t)d.T);
  size_t a_hf = take((size_t)d.G);
  size_t a_own = take((size_t)(d.T + 1) * 4);
  if (s != nullptr) {
    s->mask = reinterpret_cast<uint32_t*>(base + a_mask);
    s->mask2 = reinterpret_cast<uint32_t*>(base + a_mask2);
    s->hist = reinterpret_cast<int32_t*>(base + a_hist);
    s->off = reinterpret_cast<int32_t*>(base + a_off);
    s->key = reinterpret_cast<int32_t*>(base + a_key);
    s->pos = reinterpret_cast<int32_t*>(base + a_pos);
    s->warp_cnt = reinterpret_cast<int32_t*>(base + a_wc);
    s->scan_tot = reinterpret_cast<int32_t*>(base + a_st);
    s->idx = n_idx ? reinterpret_cast<int32_t*>(base + a_idx) : nullptr;
    s->state = base + a_state;
    s->cls = base + a_cls;
    s->has_first = base + a_hf;
    s->own = reinterpret_cast<int32_t*>(base + a_own);
  }
  return o;
}

size_t select_smem_bytes(Dims d) { return sel_smem_layout(d, nullptr, nullptr); }

__device__ __forceinline__ bool is_decoded(uint8_t s) { return s == TEAM_TOK_NEW || s == TEAM_TOK_CACHED; }

__global__ void __launch_bounds__(kSelThreads, 1)
k_select(const float* __restrict__ logits, StepPtrs st, Workspace ws, RoutePtrs ex, Dims d, Policy p, int item_tile,
         int wait_prior, int mode, int skip_dispatch) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  SelSmem s;
  sel_smem_layout(d, &s, smem_raw);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int T = d.T, E = d.E, k = d.k, ns = d.ns, EN = d.E + d.ns;
  // the expert kernel may be scheduled now: its prologue overlaps this kernel and it waits for this grid's end
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int n_words32 = 8;
  RoutePtrs& r = ws.r;
  const int S = T * k;
  // warps taking part in the dispatch walk: enough for 32 slots each, so small steps scan little
  const int nw = min(kSelWarps, (S + 31) / 32);
  // kSelRounds: CTA b of the grid routes the rows of the groups g with g % gridDim.x == b (the necessary set
  // E_A is per group, so groups are independent up to the dispatch); every CTA classifies all rows.
  // kSelCluster: the grid is one thread-block cluster; CTA b routes a contiguous block of ceil(T / C) rows
  // (routing 32 rows at once is bound by one SM's issue rate, so the rows are spread over SMs), the CTAs'
  // partial E_A sets are united through distributed shared memory between the rounds, and CTA 0 goes on to the
  // dispatch.
  const int nb = gridDim.x, cta = blockIdx.x;
  const int rows_per_cta = mode == kSelCluster ? (T + nb - 1) / nb : T;
  const int t0 = mode == kSelCluster ? min(T, cta * rows_per_cta) : 0, t1 = min(T, t0 + rows_per_cta);
  auto own_row = [&](int t) {
    if (mode == kSelRounds) return (s.key[t] >> 8) % nb == cta;
    return t >= t0 && t < t1;
  };
  // at most one row per warp: the row's logits are fetched once and stay in registers through both rounds
  const bool one_row_per_warp = (mode == kSelAll || mode == kSelCluster) && t1 - t0 <= kSelWarps;

  // ---- stage the step state (inputs of the call, not produced by the preceding kernel) ---------
  for (int i = tid; i < d.G * n_words32; i += kSelThreads) s.mask[i] = 0u;
  for (int i = tid; i < d.G; i += kSelThreads) s.has_first[i] = 0;
  if (tid == 0) s.own[T] = 0;
  for (int i = tid; i < nw * EN; i += kSelThreads) s.hist[i] = 0;
  float conf_r[TEAM_MAX_ROWS / kSelThreads];     // confidences of the rows this thread classifies, fetched with the rest
#pragma unroll
  for (int i = 0; i < TEAM_MAX_ROWS / kSelThreads; ++i) {
    const int t = tid + i * kSelThreads;
    conf_r[i] = t < T ? st.conf[t] : 0.f;
  }
  for (int t = tid; t < T && mode != kSelDispatch; t += kSelThreads) {
    int g = st.group[t], b = st.branch[t];
    if (g < 0 || g >= d.G || b < 0 || b > 255) {
      set_status(ws.status, TEAM_ERR_STATE, 1);
      g = min(max(g, 0), d.G - 1);
      b = min(max(b, 0), 255);
    }
    s.key[t] = g * 256 + b;
    s.pos[t] = st.pos[t];
    s.state[t] = st.tok_state[t];
  }
  __syncthreads();

  // ---- Eq. 4: classification --------------------------------------------------------------
  for (int t = tid; t < T && mode != kSelDispatch; t += kSelThreads) {
    const uint8_t state = s.state[t];
    uint8_t c;
    if (state == TEAM_TOK_CACHED) {
      c = (p.flags & TEAM_F_DCD) ? TEAM_CLS_SKIP : TEAM_CLS_FIRST;
    } else if (state == TEAM_TOK_NEW || !(p.flags & TEAM_F_LAC)) {
      c = TEAM_CLS_FIRST;
    } else {
      const int key = s.key[t], mypos = s.pos[t];
      const int lim = p.inclusive ? p.L_hot : p.L_hot - 1;   // |pos - j| <= lim
      bool hot = conf_r[t / kSelThreads] > p.tau_hot;
      if (p.prefix_decoded && mypos + 1 <= lim) hot = true;
      for (int u = t - 1; !hot && u >= 0 && s.key[u] == key; --u) {
        if (t - u > TEAM_MAX_BLOCK) { set_status(ws.status, TEAM_ERR_STATE, 2); break; }
        if (is_decoded(s.state[u]) && abs(mypos - s.pos[u]) <= lim) hot = true;
      }
      for (int u = t + 1; !hot && u < T && s.key[u] == key; ++u) {
        if (u - t > TEAM_MAX_BLOCK) { set_status(ws.status, TEAM_ERR_STATE, 2); break; }
        if (is_decoded(s.state[u]) && abs(mypos - s.pos[u]) <= lim) hot = true;
      }
      c = hot ? TEAM_CLS_FIRST : TEAM_CLS_COLD;
    }
    s.cls[t] = c;
    if (c == TEAM_CLS_FIRST) s.has_first[s.key[t] >> 8] = 1;
  }
  __syncthreads();
  // A group with no first-round row: its masked rows are all routed freely.  (Each thread only
  // rewrites rows it classified itself, so the next barrier is the one after round 1's reads.)
  for (int t = tid; t < T && mode != kSelDispatch; t += kSelThreads)
    if (s.cls[t] == TEAM_CLS_COLD && !s.has_first[s.key[t] >> 8]) s.cls[t] = TEAM_CLS_FIRST;

  // kSelRounds: the rows of this CTA's groups, listed once (in any order: rows are routed independently and E_A
  // is a union), so that the routing rounds walk 1/grid of the rows instead of testing every row in every warp
  if (mode == kSelRounds) {
    for (int t0r = 0; t0r < T; t0r += kSelThreads) {
      const int t = t0r + tid;
      const bool mine = t < T && (s.key[t] >> 8) % nb == cta;
      const unsigned bal = __ballot_sync(0xffffffffu, mine);
      int base = 0;
      if (lane == 0 && bal) base = atomicAdd(&s.own[T], __popc(bal));
      base = __shfl_sync(0xffffffffu, base, 0);
      if (mine) s.own[base + __popc(bal & ((1u << lane) - 1u))] = t;
    }
  }
  // Everything above depends on the step state only (inputs of the call) and overlaps the preceding
  // kernel of the stream; the logits come from that kernel.
  if (wait_prior) asm volatile("griddepcontrol.wait;" ::: "memory");
  // With at most one row per warp the row's logits are fetched now and stay in registers through
  // both routing rounds.
  float keep[kMaxPerLane];
  float keep_max = 0.f, keep_denom = 1.f;
  if (one_row_per_warp && t0 + warp < t1) load_row(logits + (size_t)(t0 + warp) * E, E, lane, keep, keep_max, keep_denom);
  if (mode == kSelDispatch) {
    // classes and choices were left in the routing tables by the kSelRounds grid
    for (int t = tid; t < T; t += kSelThreads) s.cls[t] = __ldcg(r.tok_class + t);
    if (s.idx)
      for (int i = tid; i < S; i += kSelThreads) s.idx[i] = __ldcg(r.topk_idx + i);
  }
  __syncthreads();

  // ---- Algorithm 1, round 1 (free top-k) then round 2 (top-k inside E_A) -------------------
  for (int round = 1; round <= 2 && mode != kSelDispatch; ++round) {
    const int n_mine = mode == kSelRounds ? s.own[T] : t1 - t0;
    for (int i = warp; i < n_mine; i += kSelWarps) {
      const int t = mode == kSelRounds ? s.own[i] : t0 + i;
      const uint8_t c = s.cls[t];
      if (round == 1 && c == TEAM_CLS_SKIP) {
        if (lane < k) {
          if (s.idx) s.idx[t * k + lane] = -1;
          r.topk_idx[t * k + lane] = -1;
          r.topk_w[t * k + lane] = 0.f;
          if (ex.topk_idx) ex.topk_idx[t * k + lane] = -1;
          if (ex.topk_w) ex.topk_w[t * k + lane] = 0.f;
        }
        if (lane == 0) {
          r.margin[t] = __builtin_huge_valf();
          if (ex.margin) ex.margin[t] = __builtin_huge_valf();
        }
        if (ex.probs)
          for (int e = lane; e < E; e += 32) ex.probs[(size_t)t * E + e] = 0.f;
        continue;
      }
      if ((round == 1 && c != TEAM_CLS_FIRST) || (round == 2 && c != TEAM_CLS_COLD)) continue;
      const int g = s.key[t] >> 8;
      float v[kMaxPerLane];
      float row_max, denom;
      if (one_row_per_warp) {
#pragma unroll
        for (int i = 0; i < kMaxPerLane; ++i) v[i] = keep[i];
        row_max = keep_max;
        denom = keep_denom;
      } else {
        load_row(logits + (size_t)t * E, E, lane, v, row_max, denom);
      }
      if (ex.probs) {
#pragma unroll
        for (int i = 0; i < kMaxPerLane; ++i) {
          const int e = i * 32 + lane;
          if (e < E) ex.probs[(size_t)t * E + e] = expf(v[i] - row_max) / denom;
        }
      }
      if (round == 2) {
#pragma unroll
        for (int i = 0; i < kMaxPerLane; ++i)
          if (!((s.mask[g * n_words32 + i] >> lane) & 1u)) v[i] = kNegInf;
      }
      TopkResult tr = warp_topk(v, k, lane, (E + 31) / 32);
      const float w = routing_weight(tr, k, lane, row_max, denom, p.norm_topk);
      if (lane < k) {
        if (s.idx) s.idx[t * k + lane] = tr.idx;
        r.topk_idx[t * k + lane] = tr.idx;
        r.topk_w[t * k + lane] = w;
        if (ex.topk_idx) ex.topk_idx[t * k + lane] = tr.idx;
        if (ex.topk_w) ex.topk_w[t * k + lane] = w;
        if (tr.idx < 0) set_status(ws.status, TEAM_ERR_STATE, 3);
        else if (round == 1) atomicOr(&s.mask[g * n_words32 + (tr.idx >> 5)], 1u << (tr.idx & 31));
      }
      if (lane == 0) {
        r.margin[t] = tr.margin;
        if (ex.margin) ex.margin[t] = tr.margin;
      }
    }
    __syncthreads();
    if (mode == kSelCluster && round == 1) {
      // every group's E_A = union of what the cluster's CTAs collected from their own first-round rows
      cg::cluster_group cluster = cg::this_cluster();
      cluster.sync();
      for (int i = tid; i < d.G * n_words32; i += kSelThreads) {
        uint32_t m = 0u;
        for (int rr = 0; rr < nb; ++rr) m |= cluster.map_shared_rank(s.mask, rr)[i];
        s.mask2[i] = m;
      }
      cluster.sync();                   // nobody reads a peer's partial set after this
      for (int i = tid; i < d.G * n_words32; i += kSelThreads) s.mask[i] = s.mask2[i];
      __syncthreads();
    }
  }
  const int32_t* idx_src = s.idx ? s.idx : r.topk_idx;

  // ---- exports that need no further work: by the upper half of the CTA, beside the dispatch below ----
  for (int t = tid - kSelThreads / 2; t >= 0 && t < T && mode != kSelDispatch; t += kSelThreads / 2) {
    if (!own_row(t)) continue;
    r.tok_class[t] = s.cls[t];
    if (ex.tok_class) ex.tok_class[t] = s.cls[t];
  }
  {
    const int n_words64 = (E + 63) / 64;
    for (int i = tid - kSelThreads / 2; i >= 0 && i < d.G * n_words64 && mode != kSelDispatch; i += kSelThreads / 2) {
      const int g = i / n_words64, wd = i % n_words64;
      if ((mode == kSelRounds && g % nb != cta) || (mode == kSelCluster && cta != 0)) continue;
      const uint64_t m = (uint64_t)s.mask[g * n_words32 + 2 * wd] | ((uint64_t)s.mask[g * n_words32 + 2 * wd + 1] << 32);
      r.group_mask[i] = m;
      if (ex.group_mask) ex.group_mask[i] = m;
    }
  }

  // The dispatch tables are skipped when nobody reads them: no export asked for, and an expert kernel that
  // works from the rows' choices alone (at most 8 rows, all resident).
  if (mode == kSelRounds || skip_dispatch) return;
  if (mode == kSelCluster) {
    // all CTAs' choices are in the routing tables and visible; CTA 0 alone builds the dispatch tables from them
    cg::this_cluster().sync();
    if (cta != 0) return;
    if (s.idx)
      for (int i = tid; i < S; i += kSelThreads) s.idx[i] = __ldcg(r.topk_idx + i);
    __syncthreads();
  }

  // ---- dispatch: stable counting sort of slots by expert ------------------------------------
  // Small steps (at most kSmallSlots routed slots): expert e's thread counts its slots by walking the
  // slot list in shared memory and, after the scan, walks it again to place them (ascending slot id).
  // Larger steps: routed slots t*k+j are walked in ascending order, warp w < nw owning a contiguous
  // range, so the rank of a slot inside its expert is (slots of that expert in earlier warps) +
  // (earlier in this warp).
  const bool small = s.idx != nullptr && S <= kSmallSlots;
  const int per_warp = ((S + nw - 1) / nw + 31) & ~31;
  const int lo = min(S, warp * per_warp), hi = warp < nw ? min(S, lo + per_warp) : lo;
  int32_t* my_hist = s.hist + (warp < nw ? warp : 0) * EN;
  if (!small) {
    for (int base = lo; base < hi; base += 32) {
      const int slot = base + lane;
      const int e = (slot < hi) ? idx_src[slot] : -1;
      const unsigned peers = __match_any_sync(0xffffffffu, e);
      if (e >= 0 && (__ffs(peers) - 1) == lane) my_hist[e] += __popc(peers);
      __syncwarp();
    }
  }
  // number of computed rows; shared experts take every one of them
  int n_rows_active = 0;
  if (T <= 32) {
    // every warp counts for itself: nothing to exchange
    n_rows_active = __popc(__ballot_sync(0xffffffffu, lane < T && s.cls[lane] != TEAM_CLS_SKIP));
  } else {
    int c = 0;
    for (int base = warp * 32; base < T; base += kSelThreads) {
      const int t = base + lane;
      const bool a = t < T && s.cls[t] != TEAM_CLS_SKIP;
      c += __popc(__ballot_sync(0xffffffffu, a));
    }
    if (lane == 0) s.warp_cnt[warp] = c;
  }
  if (!small || T > 32) __syncthreads();      // per-warp histograms and row counts are complete
  if (T > 32) {
    const int used = min(kSelWarps, (T + 31) / 32);
    for (int w = 0; w < used; ++w) n_rows_active += s.warp_cnt[w];
  }
  // ---- per-expert counts, then a scan over experts by ceil(EN / 32) warps ----------------------
  const int nwe = (EN + 31) / 32;            // EN <= 260: at most 9 warps, expert e = tid
  int c = 0, tiles = 0, incl_c = 0, incl_t = 0, arank = 0;
  unsigned act_b = 0;
  uint32_t mine[kSmallSlots / 32] = {};
  if (warp < nwe) {
    const int e = tid;
    if (e < E) {
      if (small) {
        // which of the (at most kSmallSlots) slots chose this expert: one bit per slot
#pragma unroll
        for (int q = 0; q < kSmallSlots / 32; ++q) {
          if (q * 32 < S) {
#pragma unroll
            for (int i = 0; i < 32; i += 4) {
              const int at = q * 32 + i;
              if (at < S) {
                const int4 v = *reinterpret_cast<const int4*>(s.idx + at);      // the array is padded to 16 bytes
                mine[q] |= (uint32_t)(v.x == e) << i | (uint32_t)(v.y == e && at + 1 < S) << (i + 1) |
                           (uint32_t)(v.z == e && at + 2 < S) << (i + 2) | (uint32_t)(v.w == e && at + 3 < S) << (i + 3);
              }
            }
            c += __popc(mine[q]);
          }
        }
      } else {
        // turn per-warp counts into per-warp starting ranks
        for (int w = 0; w < nw; ++w) {
          const int cw = s.hist[w * EN + e];
          s.hist[w * EN + e] = c;
          c += cw;
        }
      }
    } else if (e < EN) {
      c = n_rows_active;
    }
    tiles = (c + item_tile - 1) / item_tile;      // work items: ceil(c / item_tile) per expert ...
    if (e < E && (e < d.elo || e >= d.ehi)) tiles = 0;      // ... of this rank's own (expert parallelism)
    incl_c = c;
    incl_t = tiles;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int n1 = __shfl_up_sync(0xffffffffu, incl_c, o), n2 = __shfl_up_sync(0xffffffffu, incl_t, o);
      if (lane >= o) {
        incl_c += n1;
        incl_t += n2;
      }
    }
    act_b = __ballot_sync(0xffffffffu, c > 0);
    arank = __popc(act_b & ((1u << lane) - 1));
    if (lane == 31) {
      s.scan_tot[warp] = incl_c;
      s.scan_tot[kSelWarps + warp] = incl_t;
      s.scan_tot[2 * kSelWarps + warp] = __popc(act_b);
    }
  }
  __syncthreads();
  int total = 0;
  for (int w = 0; w < nwe; ++w) total += s.scan_tot[w];
  if (warp < nwe) {
    const int e = tid;
    int pc = 0, pt = 0, pa = 0;
    for (int w = 0; w < warp; ++w) {
      pc += s.scan_tot[w];
      pt += s.scan_tot[kSelWarps + w];
      pa += s.scan_tot[2 * kSelWarps + w];
    }
    const int excl = pc + incl_c - c, tbase = pt + incl_t - tiles;
    arank += pa;
    if (e < EN) {
      r.expert_count[e] = c;
      r.expert_offset[e] = excl;
      if (ex.expert_count) ex.expert_count[e] = c;
      if (ex.expert_offset) ex.expert_offset[e] = excl;
      if (!small) s.off[e] = excl;
      if (c > 0) {
        r.active[arank] = e;
        if (ex.active) ex.active[arank] = e;
        for (int i = 0; i < tiles; ++i) {
          WorkItem it;
          it.e = e;
          it.begin = excl + i * item_tile;
          it.n = min(item_tile, c - i * item_tile);
          it.pad = 0;
          ws.items[tbase + i] = it;
        }
        if (small) {
          // place this expert's slots: routed ones by ascending slot id, a shared expert's by ascending row
          int at = excl;
          if (e < E) {
#pragma unroll
            for (int q = 0; q < kSmallSlots / 32; ++q) {
              for (uint32_t m = mine[q]; m != 0; m &= m - 1) {
                const int slot = q * 32 + __ffs(m) - 1;
                r.perm[at] = slot;
                if (ex.perm) ex.perm[at] = slot;
                ++at;
              }
            }
          } else {
            for (int t = 0; t < T; ++t) {
              if (s.cls[t] != TEAM_CLS_SKIP) {
                const int slot = T * k + (e - E) * T + t;
                r.perm[at] = slot;
                if (ex.perm) ex.perm[at] = slot;
                ++at;
              }
            }
          }
        }
      }
    }
    if (warp == nwe - 1) {
      // inactive tail of the active list, and the totals
      const int n_act = pa + __popc(act_b), n_items = pt + __shfl_sync(0xffffffffu, incl_t, 31);
      for (int i = n_act + lane; i < EN; i += 32) {
        r.active[i] = -1;
        if (ex.active) ex.active[i] = -1;
      }
      if (lane == 0) {
        r.expert_offset[EN] = total;
        if (ex.expert_offset) ex.expert_offset[EN] = total;
        *r.n_active = n_act;
        *r.n_rows_active = n_rows_active;
        *ws.n_items = n_items;
        if (ex.n_active) *ex.n_active = n_act;
        if (ex.n_rows_active) *ex.n_rows_active = n_rows_active;
      }
    }
  }
  if (!small) {
    __syncthreads();
    // second walk: place the routed slots
    for (int base = lo; base < hi; base += 32) {
      const int slot = base + lane;
      const int e = (slot < hi) ? idx_src[slot] : -1;
      const unsigned peers = __match_any_sync(0xffffffffu, e);
      if (e >= 0) {
        const int rank = my_hist[e] + __popc(peers & ((1u << lane) - 1));
        const int at = s.off[e] + rank;
        r.perm[at] = slot;
        if (ex.perm) ex.perm[at] = slot;
      }
      __syncwarp();
      if (e >= 0 && (__ffs(peers) - 1) == lane) my_hist[e] += __popc(peers);
      __syncwarp();
    }
    // shared experts: slot T*k + s*T + t for every active row t, ascending t.
    if (ns > 0 && warp == kSelWarps - 1) {
      int run = 0;
      for (int base = 0; base < T; base += 32) {
        const int t = base + lane;
        const bool a = t < T && s.cls[t] != TEAM_CLS_SKIP;
        const unsigned b = __ballot_sync(0xffffffffu, a);
        if (a) {
          const int rank = run + __popc(b & ((1u << lane) - 1));
          for (int sh = 0; sh < ns; ++sh) {
            const int at = s.off[E + sh] + rank;
            const int slot = T * k + sh * T + t;
            r.perm[at] = slot;
            if (ex.perm) ex.perm[at] = slot;
          }
        }
        run += __popc(b);
      }
    }
  }
  // unused tail of perm
  for (int i = total + tid; i < T * (k + ns); i += kSelThreads) {
    r.perm[i] = -1;
    if (ex.perm) ex.perm[i] = -1;
  }
}

// The opt-in is per device and shared by all contexts: it is only ever raised.
cudaError_t configure_select(Dims max_dims) {
  static std::mutex mu;
  static int prepared[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const int smem = (int)select_smem_bytes(max_dims);
  std::lock_guard<std::mutex> lock(mu);
  if (dev >= 0 && dev < 64 && prepared[dev] >= smem && prepared[dev] > 0) return cudaSuccess;
  e = cudaFuncSetAttribute(k_select, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  // same carve-out as the expert kernel that follows: no reconfiguration of the SM in between
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(k_select, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
  if (e == cudaSuccess && dev >= 0 && dev < 64) prepared[dev] = smem;
  return e;
}

cudaError_t launch_select(const float* logits, StepPtrs st, Workspace ws, RoutePtrs ex, Dims d, Policy p,
                          int item_tile, bool need_tables, cudaStream_t s) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(1);
  cfg.blockDim = dim3(kSelThreads);
  cfg.dynamicSmemBytes = select_smem_bytes(d);
  cfg.stream = s;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;   // staging the step state overlaps the router kernel
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  // Several groups and more rows than one CTA routes at once (one row per warp): the routing rounds run as
  // one CTA per group (up to 32), the dispatch as a second single-CTA launch.
  const int group_ctas = d.G < 128 ? d.G : 128;
  if (d.T > kSelWarps && (d.G == 1 || d.T / group_ctas > kSelWarps)) {
    // one group, or groups of more rows than a CTA routes at once: one cluster, rows split over its CTAs
    const int c = d.T > 64 ? 8 : 4;        // 16 rows or fewer per CTA up to 128 rows
    cfg.gridDim = dim3(c);
    cudaLaunchAttribute attrs[2];
    attrs[0] = attr;
    attrs[1].id = cudaLaunchAttributeClusterDimension;
    attrs[1].val.clusterDim.x = c;
    attrs[1].val.clusterDim.y = 1;
    attrs[1].val.clusterDim.z = 1;
    cfg.attrs = attrs;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, k_select, logits, st, ws, ex, d, p, item_tile, 1, (int)kSelCluster, 0);
  }
  if (d.G > 1 && d.T > kSelWarps) {
    cfg.gridDim = dim3(group_ctas);
    cudaError_t e = cudaLaunchKernelEx(&cfg, k_select, logits, st, ws, ex, d, p, item_tile, 1, (int)kSelRounds, 0);
    if (e != cudaSuccess) return e;
    cfg.gridDim = dim3(1);
    return cudaLaunchKernelEx(&cfg, k_select, logits, st, ws, ex, d, p, item_tile, 1, (int)kSelDispatch, 0);
  }
  return cudaLaunchKernelEx(&cfg, k_select, logits, st, ws, ex, d, p, item_tile, 1, (int)kSelAll, need_tables ? 0 : 1);
}

int select_launches(Dims d) {
  const int group_ctas = d.G < 128 ? d.G : 128;
  if (d.T > kSelWarps && (d.G == 1 || d.T / group_ctas > kSelWarps)) return 1;
  return d.G > 1 && d.T > kSelWarps ? 2 : 1;
}

}  // namespace team
