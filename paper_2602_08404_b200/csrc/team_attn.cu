// The attention half of delayed caching (Sec. 4.1; block diffusion, Sec. 2): attention of the block being decoded
// -- bidirectional inside the block, over the cached keys / values of earlier blocks (the prefix) -- where the rows
// of cached tokens are not computed and their keys / values come from an in-block cache, followed by the delayed
// insertion of the newly accepted tokens' keys / values into that cache.
//
// team_block_attention runs head size 128 on the tensor-memory kernel of team_attn_tc.cu and head size 64 on
// k_block_attention below.
// k_block_attention: a contraction, so it runs on the tensor cores.  The (computed row, query head) pairs that share
// one (sequence, branch) and one key / value head are the M side: a CTA owns 128 of them (8 warps x 16), their
// queries live in registers as A fragments.  Keys and values are walked in tiles of 64 (prefix first, then the
// block's positions: the fresh key of a computed row, the cached one otherwise) through a three-stage cp.async ring
// in shared memory (16-byte pieces, xor-swizzled so that ldmatrix is conflict-free).  Per tile a warp forms
// S = Q K^T with mma.sync (bf16 in, fp32 out), updates the running maximum and sum of its rows (online softmax, in
// base 2), and adds P V into its fp32 output fragments; P goes in as a bf16 pair hi + lo so that the product keeps
// fp32-like accuracy.  The keys of one M tile are split over the CTAs of a thread-block cluster (1, 2, 4 or 8, chosen
// so that the grid fills the SMs); at the end every CTA leaves its partial (max, sum, output) in its own shared
// memory and rank z of the cluster merges rows z*128/n .. of all partials through distributed shared memory and
// writes them: no scratch buffer in global memory, no second kernel.
// k_attn_insert: after the pass, the fresh key / value of every decoded row computed in the base branch goes into
// the in-block cache at its position.
#include <cooperative_groups.h>

#include <mutex>

#include "team_attn.cuh"
#include "team_topk.cuh"

namespace cg = cooperative_groups;

namespace team {

constexpr int kAttnThreads = 256;
constexpr int kAttnWarps = 8;
constexpr int kAttnKeys = 64;          // keys per tile
constexpr int kAttnStages = 3;

__device__ __forceinline__ void at_cp16(uint32_t dst, const void* src, int bytes) {   // bytes 0: zero fill
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void at_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void at_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void at_ldsm4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void at_ldsm4t(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// no "volatile": a pure function of its registers, so the scheduler may interleave independent accumulators
__device__ __forceinline__ void at_mma(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float at_exp2(float x) {       // 2^x, relative error 2^-22; -inf -> 0
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// p as a bf16 pair: hi = rn(p), lo = rn(p - hi); two probabilities per register (low half = the lower key)
__device__ __forceinline__ void at_split(float p0, float p1, uint32_t& hi, uint32_t& lo) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(p0, p1);
  const float2 hf = __bfloat1622float2(h);
  const __nv_bfloat162 l = __floats2bfloat162_rn(p0 - hf.x, p1 - hf.y);
  hi = *reinterpret_cast<const uint32_t*>(&h);
  lo = *reinterpret_cast<const uint32_t*>(&l);
}

template <int D>
__global__ void __launch_bounds__(kAttnThreads, 1) k_block_attention(AttnArgs a, int n_splits) {
  extern __shared__ __align__(128) unsigned char attn_smem[];
  constexpr int ROWB = D * 2;                               // bytes of one staged key / value row
  constexpr int TILEB = kAttnKeys * ROWB;                   // one K (or V) tile
  constexpr int KS = D / 16;                                // k-steps of Q K^T
  constexpr int OSTRIDE = D + 8;                            // floats per row of the partial output (padded)
  __shared__ int s_comp[TEAM_MAX_BLOCK], s_list[TEAM_MAX_BLOCK], s_cnt[2];
  __shared__ float s_m[kAttnPairs], s_l[kAttnPairs];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int m_tile = blockIdx.x, run = blockIdx.y / a.Hkv, g = blockIdx.y - run * a.Hkv, z = blockIdx.z;
  const int L = a.L, rep = a.Hq / a.Hkv;
  const int row0 = run * L, s = run / a.B;
  // ---- the run's rows: layout contract, which of them are computed ----
  bool comp = false;
  unsigned bal = 0u;
  if (tid < TEAM_MAX_BLOCK) {                               // two warps cover the block's positions
    if (tid < L) {
      const int t = row0 + tid;
      const bool ok = a.pos[t] == tid && a.group[t] == s && a.branch[t] == run % a.B;
      if (!ok && a.status != nullptr) set_status(a.status, TEAM_ERR_STATE, 40);
      comp = attn_computed(a.tok_state[t], a.flags);
      s_comp[tid] = comp ? 1 : 0;
    }
    bal = __ballot_sync(0xffffffffu, comp);
    if (lane == 0) s_cnt[warp] = __popc(bal);
  }
  __syncthreads();
  if (comp) s_list[(warp ? s_cnt[0] : 0) + __popc(bal & ((1u << lane) - 1u))] = tid;
  __syncthreads();
  const int n_pairs = (s_cnt[0] + s_cnt[1]) * rep;
  if (m_tile * kAttnPairs >= n_pairs) return;               // the whole cluster shares (m_tile, run): it leaves together
  const int plen = min(max(a.prefix_len[s], 0), a.P);
  const int n_keys = plen + L;
  const int tiles_total = (n_keys + kAttnKeys - 1) / kAttnKeys;
  const int tps = (tiles_total + n_splits - 1) / n_splits;
  const int t_begin = min(z * tps, tiles_total), t_end = min(t_begin + tps, tiles_total);
  const bool warp_active = m_tile * kAttnPairs + warp * 16 < n_pairs;
  // ---- this thread's two pairs (fragment rows lane/4 and lane/4 + 8) and their queries as A fragments ----
  uint32_t qf[KS][4];
  {
    const __nv_bfloat16* qp[2];
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
      const int gp = m_tile * kAttnPairs + warp * 16 + (lane >> 2) + hh * 8;
      qp[hh] = nullptr;
      if (gp < n_pairs) {
        const int c = gp / rep, j = gp - c * rep;
        qp[hh] = a.q + ((size_t)(row0 + s_list[c]) * a.Hq + g * rep + j) * D + (lane & 3) * 2;
      }
    }
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      qf[ks][0] = qp[0] ? *reinterpret_cast<const uint32_t*>(qp[0] + ks * 16) : 0u;
      qf[ks][1] = qp[1] ? *reinterpret_cast<const uint32_t*>(qp[1] + ks * 16) : 0u;
      qf[ks][2] = qp[0] ? *reinterpret_cast<const uint32_t*>(qp[0] + ks * 16 + 8) : 0u;
      qf[ks][3] = qp[1] ? *reinterpret_cast<const uint32_t*>(qp[1] + ks * 16 + 8) : 0u;
    }
  }
  // ---- tile loads: thread -> key tid / 4 of the tile, pieces (tid & 3) + 4 i ----
  const uint32_t smem0 = (uint32_t)__cvta_generic_to_shared(attn_smem);
  auto issue_tile = [&](int t, int stage) {
    const int j = tid >> 2, key = t * kAttnKeys + j;
    const __nv_bfloat16 *ks_ = a.k_prefix, *vs_ = a.v_prefix;
    int bytes = 0;
    if (key < n_keys) {
      bytes = 16;
      size_t o;
      if (key < plen) {
        o = (((size_t)s * a.P + key) * a.Hkv + g) * D;
      } else {
        const int p = key - plen;
        if (s_comp[p]) {
          o = ((size_t)(row0 + p) * a.Hkv + g) * D;
          ks_ = a.k_new; vs_ = a.v_new;
        } else {
          o = (((size_t)s * L + p) * a.Hkv + g) * D;
          ks_ = a.k_block; vs_ = a.v_block;
        }
      }
      ks_ += o; vs_ += o;
    }
    const uint32_t kd = smem0 + stage * (2 * TILEB) + j * ROWB, vd = kd + TILEB;
#pragma unroll
    for (int i = 0; i < D / 32; ++i) {
      const int pc = (tid & 3) + 4 * i;
      const uint32_t off = (uint32_t)((pc ^ (j & 7)) << 4);
      at_cp16(kd + off, bytes ? ks_ + pc * 8 : ks_, bytes);
      at_cp16(vd + off, bytes ? vs_ + pc * 8 : vs_, bytes);
    }
  };
#pragma unroll
  for (int i = 0; i < kAttnStages - 1; ++i) {
    if (t_begin + i < t_end) issue_tile(t_begin + i, i);
    at_commit();
  }
  // ---- the walk over this CTA's tiles ----
  const float sl2 = rsqrtf((float)D) * 1.4426950408889634f;  // scores in base 2
  float m_run[2] = {kNegInf, kNegInf}, l_run[2] = {0.f, 0.f};
  float o[D / 8][4];
#pragma unroll
  for (int i = 0; i < D / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
  // ldmatrix lane roles
  const uint32_t k_key = ((lane >> 4) & 1) * 8 + (lane & 7), k_chunk = (lane >> 3) & 1;
  const uint32_t v_key = ((lane >> 3) & 1) * 8 + (lane & 7), v_chunk = (lane >> 4) & 1;
  const uint32_t swz = lane & 7;
  for (int t = t_begin; t < t_end; ++t) {
    const int stage = (t - t_begin) % kAttnStages;
    at_wait<kAttnStages - 2>();
    __syncthreads();                                       // tile t landed; the stage of tile t-1 is free
    if (t + kAttnStages - 1 < t_end) issue_tile(t + kAttnStages - 1, (t - t_begin + kAttnStages - 1) % kAttnStages);
    at_commit();
    if (!warp_active) continue;
    const uint32_t kb = smem0 + stage * (2 * TILEB), vb = kb + TILEB;
    float sf[kAttnKeys / 8][4];
#pragma unroll
    for (int i = 0; i < kAttnKeys / 8; ++i) sf[i][0] = sf[i][1] = sf[i][2] = sf[i][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
      for (int np = 0; np < kAttnKeys / 16; ++np) {
        uint32_t b[4];
        at_ldsm4(kb + (np * 16 + k_key) * ROWB + (((2 * ks + k_chunk) ^ swz) << 4), b);
        at_mma(sf[2 * np], qf[ks], b[0], b[1]);
        at_mma(sf[2 * np + 1], qf[ks], b[2], b[3]);
      }
    }
    // scale, mask the keys past the end (last tile only), running maximum
    const int key0 = t * kAttnKeys + (lane & 3) * 2;
    const bool ragged = (t + 1) * kAttnKeys > n_keys;
    float tmax[2] = {kNegInf, kNegInf};
#pragma unroll
    for (int i = 0; i < kAttnKeys / 8; ++i) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float v = sf[i][e] * sl2;
        if (ragged && key0 + i * 8 + (e & 1) >= n_keys) v = kNegInf;
        sf[i][e] = v;
        tmax[e >> 1] = fmaxf(tmax[e >> 1], v);
      }
    }
    float corr[2];
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
      tmax[hh] = fmaxf(tmax[hh], __shfl_xor_sync(0xffffffffu, tmax[hh], 1));
      tmax[hh] = fmaxf(tmax[hh], __shfl_xor_sync(0xffffffffu, tmax[hh], 2));
      const float m_new = fmaxf(m_run[hh], tmax[hh]);      // finite: every tile holds at least one real key
      corr[hh] = at_exp2(m_run[hh] - m_new);                 // 0 on the first tile
      m_run[hh] = m_new;
      l_run[hh] *= corr[hh];
    }
#pragma unroll
    for (int i = 0; i < kAttnKeys / 8; ++i) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float p = at_exp2(sf[i][e] - m_run[e >> 1]);
        sf[i][e] = p;
        l_run[e >> 1] += p;
      }
    }
#pragma unroll
    for (int i = 0; i < D / 8; ++i) {
      o[i][0] *= corr[0]; o[i][1] *= corr[0]; o[i][2] *= corr[1]; o[i][3] *= corr[1];
    }
    // O += P V, P as hi + lo
#pragma unroll
    for (int kk = 0; kk < kAttnKeys / 16; ++kk) {
      uint32_t ph[4], pl[4];
      at_split(sf[2 * kk][0], sf[2 * kk][1], ph[0], pl[0]);
      at_split(sf[2 * kk][2], sf[2 * kk][3], ph[1], pl[1]);
      at_split(sf[2 * kk + 1][0], sf[2 * kk + 1][1], ph[2], pl[2]);
      at_split(sf[2 * kk + 1][2], sf[2 * kk + 1][3], ph[3], pl[3]);
#pragma unroll
      for (int dp = 0; dp < D / 16; dp += 2) {             // four output tiles per group: dependent MMAs four apart
        uint32_t b0[4], b1[4];
        at_ldsm4t(vb + (kk * 16 + v_key) * ROWB + (((2 * dp + v_chunk) ^ swz) << 4), b0);
        at_ldsm4t(vb + (kk * 16 + v_key) * ROWB + (((2 * dp + 2 + v_chunk) ^ swz) << 4), b1);
        at_mma(o[2 * dp], ph, b0[0], b0[1]);
        at_mma(o[2 * dp + 1], ph, b0[2], b0[3]);
        at_mma(o[2 * dp + 2], ph, b1[0], b1[1]);
        at_mma(o[2 * dp + 3], ph, b1[2], b1[3]);
        at_mma(o[2 * dp], pl, b0[0], b0[1]);
        at_mma(o[2 * dp + 1], pl, b0[2], b0[3]);
        at_mma(o[2 * dp + 2], pl, b1[0], b1[1]);
        at_mma(o[2 * dp + 3], pl, b1[2], b1[3]);
      }
    }
  }
  at_wait<0>();
  __syncthreads();                                         // every warp is done with the stages: reuse them
  // ---- this CTA's partial result into its shared memory ----
  float* s_o = reinterpret_cast<float*>(attn_smem);         // [128][OSTRIDE]
#pragma unroll
  for (int hh = 0; hh < 2; ++hh) {
    l_run[hh] += __shfl_xor_sync(0xffffffffu, l_run[hh], 1);
    l_run[hh] += __shfl_xor_sync(0xffffffffu, l_run[hh], 2);
    const int pr = warp * 16 + (lane >> 2) + hh * 8;
    if ((lane & 3) == 0) {
      s_m[pr] = m_run[hh];
      s_l[pr] = l_run[hh];
    }
    float* orow = s_o + pr * OSTRIDE + (lane & 3) * 2;
#pragma unroll
    for (int i = 0; i < D / 8; ++i) *reinterpret_cast<float2*>(orow + i * 8) = make_float2(o[i][2 * hh], o[i][2 * hh + 1]);
  }
  cg::cluster_group cluster = cg::this_cluster();
  cluster.sync();
  // ---- rank z merges rows z * R .. z * R + R - 1 of all partials (distributed shared memory) and writes them ----
  {
    constexpr int TPR = D / 4;                              // threads per row (one float4 each)
    const int R = kAttnPairs / n_splits;
    const int c4 = tid % TPR;
    for (int i = tid / TPR; i < R; i += kAttnThreads / TPR) {
      const int pr = z * R + i, gp = m_tile * kAttnPairs + pr;
      if (gp >= n_pairs) continue;
      float mk[kAttnMaxSplits], mx = kNegInf;
#pragma unroll
      for (int k = 0; k < kAttnMaxSplits; ++k) {
        mk[k] = kNegInf;
        if (k < n_splits) mk[k] = *cluster.map_shared_rank(&s_m[pr], k);
        mx = fmaxf(mx, mk[k]);
      }
      float den = 0.f;
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int k = 0; k < kAttnMaxSplits; ++k) {
        if (k >= n_splits) break;
        const float f = exp2f(mk[k] - mx);                   // 0 for a split without keys (its maximum is -inf)
        den = fmaf(f, *cluster.map_shared_rank(&s_l[pr], k), den);
        const float4 v = *reinterpret_cast<const float4*>(cluster.map_shared_rank(s_o + pr * OSTRIDE + c4 * 4, k));
        acc.x = fmaf(f, v.x, acc.x); acc.y = fmaf(f, v.y, acc.y); acc.z = fmaf(f, v.z, acc.z); acc.w = fmaf(f, v.w, acc.w);
      }
      const int c = gp / rep, j = gp - c * rep;
      float* dst = a.out + ((size_t)(row0 + s_list[c]) * a.Hq + g * rep + j) * D + c4 * 4;
      const float inv = 1.f / den;
      *reinterpret_cast<float4*>(dst) = make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
    }
  }
  cluster.sync();                                          // peers may still be reading this CTA's partial
}

// Delayed insertion (Sec. 4.1): decoded rows computed in the base branch enter the in-block cache after the pass.
__global__ void __launch_bounds__(256) k_attn_insert(AttnArgs a) {
  const int pieces = a.Hkv * a.d / 8, T = a.S * a.B * a.L;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < T * pieces; i += gridDim.x * blockDim.x) {
    const int t = i / pieces, pc = i - t * pieces;
    const int st = a.tok_state[t];
    if (!attn_computed(st, a.flags) || a.branch[t] != 0 || st == TEAM_TOK_MASKED) continue;
    if ((unsigned)a.group[t] >= (unsigned)a.S || (unsigned)a.pos[t] >= (unsigned)a.L) continue;   // reported by the attention kernel
    const size_t dst = (((size_t)a.group[t] * a.L + a.pos[t]) * a.Hkv * a.d) / 8 + pc;
    const size_t src = ((size_t)t * a.Hkv * a.d) / 8 + pc;
    reinterpret_cast<uint4*>(a.k_block)[dst] = reinterpret_cast<const uint4*>(a.k_new)[src];
    reinterpret_cast<uint4*>(a.v_block)[dst] = reinterpret_cast<const uint4*>(a.v_new)[src];
  }
}

static size_t attn_smem_bytes(int d) {
  const size_t stages = (size_t)kAttnStages * 2 * kAttnKeys * d * 2, partial = (size_t)kAttnPairs * (d + 8) * 4;
  return stages > partial ? stages : partial;
}

// per device: the dynamic shared memory opt-in of both instantiations and the SM count
static cudaError_t configure_attn(int* n_sms) {
  static std::mutex mu;
  static int sms[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  std::lock_guard<std::mutex> lock(mu);
  if (dev >= 0 && dev < 64 && sms[dev] > 0) {
    *n_sms = sms[dev];
    return cudaSuccess;
  }
  e = cudaFuncSetAttribute(k_block_attention<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attn_smem_bytes(64));
  int n = 0;
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  if (dev >= 0 && dev < 64) sms[dev] = n;
  *n_sms = n;
  return cudaSuccess;
}

}  // namespace team

extern "C" int team_block_attention(const team_attn_config* cfg, const team_step_state* st, const void* q, const void* k_new,
                                    const void* v_new, const void* k_prefix, const void* v_prefix, const int32_t* prefix_len,
                                    void* k_block, void* v_block, float* out, int32_t* status, void* stream) {
  if (cfg == nullptr || st == nullptr || !q || !k_new || !v_new || !k_prefix || !v_prefix || !prefix_len || !k_block ||
      !v_block || !out)
    return TEAM_ERR_ARG;
  if (!st->tok_state || !st->pos || !st->group || !st->branch) return TEAM_ERR_ARG;
  if (cfg->head_dim != 64 && cfg->head_dim != 128) return TEAM_ERR_SHAPE;
  if (cfg->n_heads < 1 || cfg->n_kv_heads < 1 || cfg->n_heads % cfg->n_kv_heads) return TEAM_ERR_SHAPE;
  if (cfg->block < 1 || cfg->block > TEAM_MAX_BLOCK || cfg->n_seqs < 1 || cfg->n_branches < 1 || cfg->max_prefix < 0)
    return TEAM_ERR_SHAPE;
  if ((long long)cfg->n_seqs * cfg->n_branches * cfg->n_kv_heads > 65535) return TEAM_ERR_SHAPE;
  if (st->n_rows != cfg->n_seqs * cfg->n_branches * cfg->block) return TEAM_ERR_ARG;
  const void* ptrs[] = {q, k_new, v_new, k_prefix, v_prefix, k_block, v_block, out};
  for (const void* p : ptrs)
    if ((uintptr_t)p & 15) return TEAM_ERR_ARG;
  team::AttnArgs a;
  a.q = static_cast<const __nv_bfloat16*>(q);
  a.k_new = static_cast<const __nv_bfloat16*>(k_new);
  a.v_new = static_cast<const __nv_bfloat16*>(v_new);
  a.k_prefix = static_cast<const __nv_bfloat16*>(k_prefix);
  a.v_prefix = static_cast<const __nv_bfloat16*>(v_prefix);
  a.prefix_len = prefix_len;
  a.k_block = static_cast<__nv_bfloat16*>(k_block);
  a.v_block = static_cast<__nv_bfloat16*>(v_block);
  a.tok_state = st->tok_state; a.pos = st->pos; a.group = st->group; a.branch = st->branch;
  a.out = out;
  a.status = status;
  a.S = cfg->n_seqs; a.B = cfg->n_branches; a.L = cfg->block; a.Hq = cfg->n_heads; a.Hkv = cfg->n_kv_heads;
  a.d = cfg->head_dim; a.P = cfg->max_prefix; a.flags = cfg->flags;
  int n_sms = 0;
  if (team::configure_attn(&n_sms) != cudaSuccess) {
    cudaGetLastError();
    return TEAM_ERR_CUDA;
  }
  // M tiles by the largest number of pairs a run can have; key splits (the cluster) until the grid fills the SMs,
  // each split keeping at least two tiles of the longest prefix
  const int rep = a.Hq / a.Hkv;
  const int m_tiles = (a.L * rep + team::kAttnPairs - 1) / team::kAttnPairs;
  const long long units = (long long)m_tiles * a.S * a.B * a.Hkv;
  const int tiles_max = (a.P + a.L + team::kAttnKeys - 1) / team::kAttnKeys;
  int n_splits = 1;
  while (n_splits < team::kAttnMaxSplits && units * n_splits * 2 <= n_sms && tiles_max >= 4 * n_splits) n_splits *= 2;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(m_tiles, a.S * a.B * a.Hkv, n_splits);
  lc.blockDim = dim3(team::kAttnThreads);
  lc.dynamicSmemBytes = team::attn_smem_bytes(a.d);
  lc.stream = s;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = 1; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = n_splits;
  lc.attrs = at;
  lc.numAttrs = 1;
  // head size 128: the tensor-memory kernel; head size 64: the fragment kernel
  cudaError_t e;
  if (a.d == 128) {
    e = team::configure_attention_tc();
    if (e == cudaSuccess) e = team::launch_attention_tc(a, m_tiles, n_splits, s);
  } else {
    e = cudaLaunchKernelEx(&lc, team::k_block_attention<64>, a, n_splits);
  }
  if (e != cudaSuccess) {
    cudaGetLastError();
    return TEAM_ERR_CUDA;
  }
  const int T = a.S * a.B * a.L, pieces = a.Hkv * a.d / 8;
  const int blocks = (T * pieces + 255) / 256;
  team::k_attn_insert<<<blocks < 1184 ? blocks : 1184, 256, 0, s>>>(a);
  return cudaGetLastError() == cudaSuccess ? TEAM_OK : TEAM_ERR_CUDA;
}
