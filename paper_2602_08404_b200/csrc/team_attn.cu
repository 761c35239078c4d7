// The attention half of delayed caching (Sec. 4.1; block diffusion, Sec. 2): attention of the block being decoded
// -- bidirectional inside the block, over the cached keys / values of earlier blocks (the prefix) -- where the rows
// of cached tokens are not computed and their keys / values come from an in-block cache, followed by the delayed
// insertion of the newly accepted tokens' keys / values into that cache.
//
// k_block_attention: one CTA per (sequence, branch, query head), 8 warps.  The queries of the run's computed rows
// sit in shared memory as fp32; keys and values are walked in tiles of 32 (prefix first, then the block's positions:
// the fresh key of a computed row, the cached one otherwise), staged in shared memory as bf16.  Inside a tile lane =
// key: every lane forms the whole q.k of its key (no shuffles), the row's running maximum and sum are updated
// (online softmax), and the lane that owns four output dimensions gathers p_j * v_j over the tile with one shuffle
// per key.  A warp carries up to 8 rows of the run through the tile, so a tile is read from shared memory once per
// warp, from global memory once per CTA.
// k_attn_insert: after the pass, the fresh key / value of every decoded row computed in the base branch goes into
// the in-block cache at its position.
#include <mutex>

#include "team_common.cuh"
#include "team_topk.cuh"

namespace team {

constexpr int kAttnThreads = 256;
constexpr int kAttnWarps = 8;
constexpr int kAttnTile = 32;          // keys per tile
constexpr int kAttnMaxRowsPerWarp = TEAM_MAX_BLOCK / kAttnWarps;   // 8

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

template <int D>
__global__ void __launch_bounds__(kAttnThreads) k_block_attention(AttnArgs a) {
  extern __shared__ __align__(16) unsigned char attn_smem[];
  constexpr int KSTRIDE = D * 2 + 16;                       // bytes per staged key row (padded: no bank conflicts)
  constexpr int DPL = D / 32;                               // output dimensions per lane
  float* s_q = reinterpret_cast<float*>(attn_smem);                                     // [L][D]
  unsigned char* s_k = attn_smem + (size_t)a.L * D * 4;                                   // [32][KSTRIDE]
  unsigned char* s_v = s_k + kAttnTile * KSTRIDE;                                         // [32][D * 2]
  __shared__ int s_comp[TEAM_MAX_BLOCK];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int run = blockIdx.x, h = blockIdx.y, L = a.L;
  const int row0 = run * L, s = run / a.B, g = h / (a.Hq / a.Hkv);
  // ---- the run's rows: layout contract, which of them are computed ----
  if (tid < L) {
    const int t = row0 + tid;
    const bool ok = a.pos[t] == tid && a.group[t] == s && a.branch[t] == run % a.B;
    if (!ok && a.status != nullptr) set_status(a.status, TEAM_ERR_STATE, 40);
    s_comp[tid] = attn_computed(a.tok_state[t], a.flags) ? 1 : 0;
  }
  for (int i = tid; i < L * D; i += kAttnThreads) {
    const int r = i / D, c = i - r * D;
    s_q[i] = __bfloat162float(a.q[((size_t)(row0 + r) * a.Hq + h) * D + c]);
  }
  __syncthreads();
  const int plen = min(max(a.prefix_len[s], 0), a.P);
  const int n_keys = plen + L;
  const float scale = rsqrtf((float)D);
  // this warp's rows: r = warp, warp + 8, ...
  float m[kAttnMaxRowsPerWarp], l[kAttnMaxRowsPerWarp], acc[kAttnMaxRowsPerWarp][DPL];
#pragma unroll
  for (int i = 0; i < kAttnMaxRowsPerWarp; ++i) {
    m[i] = kNegInf;
    l[i] = 0.f;
#pragma unroll
    for (int c = 0; c < DPL; ++c) acc[i][c] = 0.f;
  }
  for (int k0 = 0; k0 < n_keys; k0 += kAttnTile) {
    // ---- stage the tile: 32 keys x D bf16, 16-byte pieces ----
    constexpr int PIECES = D / 8;
    for (int i = tid; i < kAttnTile * PIECES; i += kAttnThreads) {
      const int j = i / PIECES, pc = i - j * PIECES, key = k0 + j;
      uint4 kv = make_uint4(0u, 0u, 0u, 0u), vv = make_uint4(0u, 0u, 0u, 0u);
      if (key < n_keys) {
        const __nv_bfloat16 *ks, *vs;
        if (key < plen) {
          const size_t o = (((size_t)s * a.P + key) * a.Hkv + g) * D;
          ks = a.k_prefix + o;
          vs = a.v_prefix + o;
        } else {
          const int p = key - plen;
          if (s_comp[p]) {
            const size_t o = ((size_t)(row0 + p) * a.Hkv + g) * D;
            ks = a.k_new + o;
            vs = a.v_new + o;
          } else {
            const size_t o = (((size_t)s * L + p) * a.Hkv + g) * D;
            ks = a.k_block + o;
            vs = a.v_block + o;
          }
        }
        kv = *reinterpret_cast<const uint4*>(ks + pc * 8);
        vv = *reinterpret_cast<const uint4*>(vs + pc * 8);
      }
      *reinterpret_cast<uint4*>(s_k + j * KSTRIDE + pc * 16) = kv;
      *reinterpret_cast<uint4*>(s_v + j * (D * 2) + pc * 16) = vv;
    }
    __syncthreads();
    const bool key_ok = k0 + lane < n_keys;
#pragma unroll
    for (int i = 0; i < kAttnMaxRowsPerWarp; ++i) {
      const int r = warp + i * kAttnWarps;
      if (r >= L || !s_comp[r]) continue;                  // warp-uniform
      // lane = key: the whole dot product
      float sc = 0.f;
      const float* qr = s_q + r * D;
      const unsigned char* kr = s_k + lane * KSTRIDE;
#pragma unroll
      for (int pc = 0; pc < PIECES; ++pc) {
        const uint4 kk = *reinterpret_cast<const uint4*>(kr + pc * 16);
        const float4 q0 = *reinterpret_cast<const float4*>(qr + pc * 8), q1 = *reinterpret_cast<const float4*>(qr + pc * 8 + 4);
        const float2 a0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&kk.x));
        const float2 a1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&kk.y));
        const float2 a2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&kk.z));
        const float2 a3 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&kk.w));
        sc = fmaf(q0.x, a0.x, sc); sc = fmaf(q0.y, a0.y, sc); sc = fmaf(q0.z, a1.x, sc); sc = fmaf(q0.w, a1.y, sc);
        sc = fmaf(q1.x, a2.x, sc); sc = fmaf(q1.y, a2.y, sc); sc = fmaf(q1.z, a3.x, sc); sc = fmaf(q1.w, a3.y, sc);
      }
      sc = key_ok ? sc * scale : kNegInf;
      const float m_new = fmaxf(m[i], warp_max(sc));
      const float p = key_ok ? expf(sc - m_new) : 0.f;
      const float corr = expf(m[i] - m_new);               // 0 on the first tile (m = -inf)
      l[i] = l[i] * corr + warp_sum(p);
      m[i] = m_new;
#pragma unroll
      for (int c = 0; c < DPL; ++c) acc[i][c] *= corr;
      for (int j = 0; j < kAttnTile; ++j) {
        const float pj = __shfl_sync(0xffffffffu, p, j);
        const __nv_bfloat16* vr = reinterpret_cast<const __nv_bfloat16*>(s_v + j * (D * 2)) + lane * DPL;
#pragma unroll
        for (int c = 0; c < DPL; ++c) acc[i][c] = fmaf(pj, __bfloat162float(vr[c]), acc[i][c]);
      }
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < kAttnMaxRowsPerWarp; ++i) {
    const int r = warp + i * kAttnWarps;
    if (r >= L || !s_comp[r]) continue;
    float* o = a.out + ((size_t)(row0 + r) * a.Hq + h) * D + lane * DPL;
#pragma unroll
    for (int c = 0; c < DPL; ++c) o[c] = acc[i][c] / l[i];
  }
}

// Delayed insertion (Sec. 4.1): decoded rows computed in the base branch enter the in-block cache after the pass.
__global__ void __launch_bounds__(256) k_attn_insert(AttnArgs a) {
  const int pieces = a.Hkv * a.d / 8, T = a.S * a.B * a.L;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < T * pieces; i += gridDim.x * blockDim.x) {
    const int t = i / pieces, pc = i - t * pieces;
    const int st = a.tok_state[t];
    if (!attn_computed(st, a.flags) || a.branch[t] != 0 || st == TEAM_TOK_MASKED) continue;
    const size_t dst = (((size_t)a.group[t] * a.L + a.pos[t]) * a.Hkv * a.d) / 8 + pc;
    const size_t src = ((size_t)t * a.Hkv * a.d) / 8 + pc;
    reinterpret_cast<uint4*>(a.k_block)[dst] = reinterpret_cast<const uint4*>(a.k_new)[src];
    reinterpret_cast<uint4*>(a.v_block)[dst] = reinterpret_cast<const uint4*>(a.v_new)[src];
  }
}

static size_t attn_smem_bytes(int L, int d) { return (size_t)L * d * 4 + kAttnTile * (d * 2 + 16) + kAttnTile * d * 2; }

static cudaError_t configure_attn(int d, int smem) {
  static std::mutex mu;
  static int prepared[64][2] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const int di = d == 128 ? 1 : 0;
  std::lock_guard<std::mutex> lock(mu);
  if (dev >= 0 && dev < 64 && prepared[dev][di] >= smem) return cudaSuccess;
  e = d == 128 ? cudaFuncSetAttribute(k_block_attention<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem)
               : cudaFuncSetAttribute(k_block_attention<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e == cudaSuccess && dev >= 0 && dev < 64) prepared[dev][di] = smem;
  return e;
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
  const size_t smem = team::attn_smem_bytes(a.L, a.d);
  if (team::configure_attn(a.d, (int)smem) != cudaSuccess) {
    cudaGetLastError();
    return TEAM_ERR_CUDA;
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  dim3 grid(a.S * a.B, a.Hq);
  if (a.d == 128) team::k_block_attention<128><<<grid, team::kAttnThreads, smem, s>>>(a);
  else team::k_block_attention<64><<<grid, team::kAttnThreads, smem, s>>>(a);
  if (cudaGetLastError() != cudaSuccess) return TEAM_ERR_CUDA;
  const int T = a.S * a.B * a.L, pieces = a.Hkv * a.d / 8;
  const int blocks = (T * pieces + 255) / 256;
  team::k_attn_insert<<<blocks < 1184 ? blocks : 1184, 256, 0, s>>>(a);
  return cudaGetLastError() == cudaSuccess ? TEAM_OK : TEAM_ERR_CUDA;
}
