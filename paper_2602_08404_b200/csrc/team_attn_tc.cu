// The attention half of delayed caching (Sec. 4.1; block diffusion, Sec. 2) for head size 128 on the fifth-generation
// tensor cores: S = Q K^T and O += P V are tcgen05.mma instructions with their accumulators in tensor memory.
//
// One CTA owns 128 (computed row, query head) pairs that share one (sequence, branch) and one key / value head, and a
// share of the keys (the CTAs of a thread-block cluster split the keys of one M tile and merge their partial results
// through distributed shared memory, as in the fragment kernel).  Thirteen warps, three roles:
//   warps 0-3  softmax: thread i owns pair i = lane i of tensor memory.  Per tile of 64 keys it reads its row of S,
//              keeps a running maximum that only moves when the new maximum exceeds it by 2^8 (then the output
//              accumulator in tensor memory is rescaled, which is rare after the first tiles), writes P = 2^(s - m)
//              into shared memory as a bf16 pair hi + lo (the A operand of the second product) and sums the row.
//   warp 4     issues the MMAs: S(t+1) ahead of P V(t), so the tensor core works on the next scores while the
//              softmax warps are busy with the current ones.
//   warps 5-12 loaders: keys by cp.async straight into the K-major 128-byte-swizzled operand layout; values into a
//              staging tile, which the same warps transpose with ldmatrix.trans / stmatrix into V^T (head dimension on
//              rows, keys contiguous), the K-major B operand of P V.  Source per key: prefix, fresh row or in-block
//              cache.
// Every wait is an mbarrier wait with a limit; when one runs out the CTA stops working, reports TEAM_ERR_TIMEOUT and
// still takes part in the cluster's barriers and frees its tensor memory.
#include <cooperative_groups.h>

#include <mutex>

#include "team_attn.cuh"
#include "team_tc_ptx.cuh"
#include "team_topk.cuh"

namespace cg = cooperative_groups;

namespace team {

constexpr int kAtD = 128;
constexpr int kAtKeys = 64;                 // keys per tile
constexpr int kAtLoadWarps = 8;                // a warp issues one cp.async per ~130 cycles: the loaders are many
constexpr int kAtLoadThreads = kAtLoadWarps * 32;
constexpr int kAtThreads = 160 + kAtLoadThreads;
constexpr int kAtKStages = 3, kAtVStages = 3, kAtVtStages = 2;
constexpr int kAtQBytes = kAttnPairs * kAtD * 2;             // 32 KB: two k-blocks of [128 rows][128 B]
constexpr int kAtPBytes = 2 * kAttnPairs * 128;              // hi and lo: [128 rows][128 B] each
constexpr int kAtVtBytes = kAtD * 128;                       // [128 rows (d)][64 keys]
constexpr int kAtKBytes = kAtKeys * kAtD * 2;                // two k-blocks of [64 rows][128 B]
constexpr int kAtVBytes = kAtKeys * kAtD * 2;                // staging: [64 keys][256 B], 16-byte pieces xor-swizzled
constexpr int kAtOffP = kAtQBytes, kAtOffVt = kAtOffP + kAtPBytes, kAtOffK = kAtOffVt + kAtVtStages * kAtVtBytes;
constexpr int kAtOffV = kAtOffK + kAtKStages * kAtKBytes, kAtOffBars = kAtOffV + kAtVStages * kAtVBytes;
constexpr int kAtSmemBytes = kAtOffBars + 256 + 1024;        // + barriers + slack for the 1024-byte alignment
constexpr int kAtOStride = kAtD + 8;                         // floats per row of the partial output (aliases K / V stages)
static_assert(kAttnPairs * kAtOStride * 4 <= kAtKStages * kAtKBytes + kAtVStages * kAtVBytes, "partial output must fit");
constexpr int kAtTmemCols = 256;                             // S: 2 x 64 columns, O: 128 columns
constexpr float kAtRescale = 8.f;                            // the maximum moves only when it grows by more than 2^8

__device__ __forceinline__ void at_cp16z(uint32_t dst, const void* src, int bytes) {   // bytes 0: zero fill
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
template <int N>
__device__ __forceinline__ void at_cp_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void at_ldsm4t(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void at_stsm4(uint32_t addr, const uint32_t (&r)[4]) {
  asm volatile("stmatrix.sync.aligned.m8n8.x4.shared.b16 [%0], {%1, %2, %3, %4};"
               ::"r"(addr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]) : "memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t (&r)[8]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
               ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float at_ex2(float x) {          // 2^x, relative error 2^-22; -inf -> 0
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// two probabilities as bf16 pairs hi = rn(p), lo = rn(p - hi); low half = the lower key
__device__ __forceinline__ void at_split2(float p0, float p1, uint32_t& hi, uint32_t& lo) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(p0, p1);
  const float2 hf = __bfloat1622float2(h);
  const __nv_bfloat162 l = __floats2bfloat162_rn(p0 - hf.x, p1 - hf.y);
  hi = *reinterpret_cast<const uint32_t*>(&h);
  lo = *reinterpret_cast<const uint32_t*>(&l);
}
__device__ __forceinline__ void bar_loaders() { asm volatile("bar.sync 1, %0;" ::"n"(kAtLoadThreads) : "memory"); }

__global__ void __launch_bounds__(kAtThreads, 1) k_block_attention_tc(AttnArgs a, int n_splits) {
  extern __shared__ unsigned char at_smem_raw[];
  unsigned char* smem = at_smem_raw + ((1024u - (smem_u32(at_smem_raw) & 1023u)) & 1023u);      // swizzled tiles: 1024-byte aligned
  const uint32_t sm0 = smem_u32(smem);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kAtOffBars);
  uint64_t* k_full = bars;                        // [3] loaders (one arrival per thread): the key tile has landed
  uint64_t* k_empty = k_full + kAtKStages;        // [3] MMA commit: S of that tile is done
  uint64_t* vt_full = k_empty + kAtKStages;       // [2] loader warps: V^T is written
  uint64_t* vt_empty = vt_full + kAtVtStages;     // [2] MMA commit: P V of that tile is done
  uint64_t* s_full = vt_empty + kAtVtStages;      // [2] MMA commit: the scores are in tensor memory
  uint64_t* s_empty = s_full + 2;                 // [2] softmax warps (4): the scores are in registers
  uint64_t* p_full = s_empty + 2;                 // [1] softmax warps (4): P is in shared memory, O is rescaled
  uint64_t* pv_done = p_full + 1;                 // [1] MMA commit: O holds the tiles so far
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(pv_done + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  int32_t* status_sink = reinterpret_cast<int32_t*>(tmem_slot + 2);      // [2] stands in for a null status pointer
  __shared__ int s_comp[TEAM_MAX_BLOCK], s_list[TEAM_MAX_BLOCK], s_cnt[2];
  __shared__ float s_m[kAttnPairs], s_l[kAttnPairs];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int m_tile = blockIdx.x, run = blockIdx.y / a.Hkv, g = blockIdx.y - run * a.Hkv, z = blockIdx.z;
  const int L = a.L, rep = a.Hq / a.Hkv;
  const int row0 = run * L, s = run / a.B;
  int32_t* status = a.status != nullptr ? a.status : status_sink;
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
  const int n_pairs = (s_cnt[0] + s_cnt[1]) * rep;
  if (m_tile * kAttnPairs >= n_pairs) return;               // the whole cluster shares (m_tile, run): it leaves together
  const int plen = min(max(a.prefix_len[s], 0), a.P);
  const int n_keys = plen + L;
  const int tiles_total = (n_keys + kAtKeys - 1) / kAtKeys;
  const int tps = (tiles_total + n_splits - 1) / n_splits;
  const int t_begin = min(z * tps, tiles_total), t_end = min(t_begin + tps, tiles_total);
  const int n_tiles = t_end - t_begin;
  if (tid == 0) {
    for (int i = 0; i < kAtKStages; ++i) {
      mbar_init(smem_u32(k_full + i), kAtLoadThreads);
      mbar_init(smem_u32(k_empty + i), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(vt_full + i), kAtLoadWarps);
      mbar_init(smem_u32(vt_empty + i), 1);
      mbar_init(smem_u32(s_full + i), 1);
      mbar_init(smem_u32(s_empty + i), 4);
    }
    mbar_init(smem_u32(p_full), 4);
    mbar_init(smem_u32(pv_done), 1);
    *abort_flag = 0;
    status_sink[0] = status_sink[1] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 4) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"((uint32_t)kAtTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  __syncthreads();                                          // s_list is complete
  // ---- loaders: the first two key / value tiles are requested before anything else is set up ----
  const int ltid = tid - 160, lw = warp - 5;
  constexpr int RPI = kAtLoadThreads / 16;                  // key rows covered per step of the copy loop
  const int c = ltid & 15, jr = ltid >> 4;                  // a loader thread's 16-byte piece and key row (jr + RPI i)
  // Keys and values travel through registers (16-byte loads, two tiles ahead, then 16-byte shared-memory stores):
  // cp.async tops out near 20 B per clock and SM here, a third of what one tile per microsecond needs.
  constexpr int NR = kAtKeys / RPI;                         // key rows per loader thread and tile
  uint4 kr0[NR], vr0[NR], kr1[NR], vr1[NR];                 // tiles of even / odd index
  auto load_tile = [&](int i, uint4 (&kk)[NR], uint4 (&vv)[NR]) {
#pragma unroll
    for (int r8 = 0; r8 < NR; ++r8) {
      const int key = (t_begin + i) * kAtKeys + r8 * RPI + jr;
      kk[r8] = vv[r8] = make_uint4(0u, 0u, 0u, 0u);          // keys past the end: zero rows
      if (key < n_keys) {
        const __nv_bfloat16 *ks = a.k_prefix, *vs = a.v_prefix;
        size_t o;
        if (key < plen) {
          o = (((size_t)s * a.P + key) * a.Hkv + g) * kAtD;
        } else {
          const int p = key - plen;
          if (s_comp[p]) {
            o = ((size_t)(row0 + p) * a.Hkv + g) * kAtD;
            ks = a.k_new; vs = a.v_new;
          } else {
            o = (((size_t)s * L + p) * a.Hkv + g) * kAtD;
            ks = a.k_block; vs = a.v_block;
          }
        }
        kk[r8] = __ldg(reinterpret_cast<const uint4*>(ks + o + c * 8));
        vv[r8] = __ldg(reinterpret_cast<const uint4*>(vs + o + c * 8));
      }
    }
  };
  auto store_tile = [&](int i, const uint4 (&kk)[NR], const uint4 (&vv)[NR]) {   // key stage i % 3, staging i % 3
    unsigned char* kst = smem + kAtOffK + (i % kAtKStages) * kAtKBytes;
    unsigned char* vst = smem + kAtOffV + (i % kAtVStages) * kAtVBytes;
#pragma unroll
    for (int r8 = 0; r8 < NR; ++r8) {
      const int j = r8 * RPI + jr;
      *reinterpret_cast<uint4*>(kst + (c >> 3) * (kAtKeys * 128) + sw128(j, c & 7)) = kk[r8];
      *reinterpret_cast<uint4*>(vst + j * 256 + ((c ^ (j & 7)) << 4)) = vv[r8];
    }
  };
  if (warp >= 5) {
    if (n_tiles > 0) load_tile(0, kr0, vr0);
    if (n_tiles > 1) load_tile(1, kr1, vr1);
  }
  // ---- the queries of this CTA's pairs: A operand of S = Q K^T, two k-blocks of [128 rows][128 B], swizzled ----
  for (int i = tid; i < kAttnPairs * 16 && warp < 5; i += 160) {
    const int pr = i >> 4, c = i & 15, gp = m_tile * kAttnPairs + pr;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (gp < n_pairs) {
      const int cr = gp / rep, j = gp - cr * rep;
      v = *reinterpret_cast<const uint4*>(a.q + ((size_t)(row0 + s_list[cr]) * a.Hq + g * rep + j) * kAtD + c * 8);
    }
    *reinterpret_cast<uint4*>(smem + (c >> 3) * (kAttnPairs * 128) + sw128(pr, c & 7)) = v;
  }
  fence_async_smem();                                       // generic-proxy writes, read by the tensor core
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  float m_used = kNegInf, l_run = 0.f;                      // softmax threads: running maximum in use (base 2) and row sum

  if (warp >= 5) {
    // ------------------------------ loaders ------------------------------
    bool ok = true;
    for (int i = 0; i < n_tiles; ++i) {
      // the key stage of tile i was read by S(i - 3)
      if (ok && i >= kAtKStages)
        ok = mbar_wait_warp(smem_u32(k_empty + i % kAtKStages), ((i / kAtKStages) & 1) ^ 1, abort_flag, status, 51);
      if (ok) {
        if (i & 1) {
          store_tile(i, kr1, vr1);
          if (i + 2 < n_tiles) load_tile(i + 2, kr1, vr1);
        } else {
          store_tile(i, kr0, vr0);
          if (i + 2 < n_tiles) load_tile(i + 2, kr0, vr0);
        }
      }
      fence_async_smem();                                   // generic-proxy writes, read by the tensor core
      if (ok) mbar_arrive(smem_u32(k_full + i % kAtKStages));
      bar_loaders();                                        // the staged values are complete, and every warp is done
                                                            // transposing tile i - 1
      if (ok) ok = mbar_wait_warp(smem_u32(vt_empty + (i & 1)), ((i >> 1) & 1) ^ 1, abort_flag, status, 52);
      if (ok) {
        // V^T: 8 x 8 blocks transposed on the way; the warps share the 16 head-dimension pieces
        const uint32_t vst = sm0 + kAtOffV + (i % kAtVStages) * kAtVBytes, vt = sm0 + kAtOffVt + (i & 1) * kAtVtBytes;
        const int mi = lane >> 3, r = lane & 7;
#pragma unroll
        for (int dd = 0; dd < 16 / kAtLoadWarps; ++dd) {
          const int dc = lw * (16 / kAtLoadWarps) + dd;
#pragma unroll
          for (int kb4 = 0; kb4 < 2; ++kb4) {
            uint32_t v[4];
            const int key = (kb4 * 4 + mi) * 8 + r;         // source: matrix mi = keys 8 (4 kb4 + mi) .., piece dc
            at_ldsm4t(vst + key * 256 + ((dc ^ r) << 4), v);
            at_stsm4(vt + sw128(dc * 8 + r, kb4 * 4 + mi), v);      // target: rows d = 8 dc + r, key piece 4 kb4 + mi
          }
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(vt_full + (i & 1)));
      }
    }
  } else if (warp == 4) {
    // ------------------------------ MMA issuer ------------------------------
    const uint32_t idesc_s = make_idesc_bf16(kAtKeys), idesc_o = make_idesc_bf16(kAtD);
    const uint32_t tm_o = tmem_base + 2 * kAtKeys;
    bool ok = true;
    auto issue_s = [&](int i) {
      const int st = i % kAtKStages, b = i & 1;
      if (!(ok = mbar_wait_warp(smem_u32(k_full + st), (i / kAtKStages) & 1, abort_flag, status, 53))) return;
      if (!(ok = mbar_wait_warp(smem_u32(s_empty + b), ((i >> 1) & 1) ^ 1, abort_flag, status, 54))) return;
      tc_fence_after();
      const uint32_t kst = sm0 + kAtOffK + st * kAtKBytes;
#pragma unroll
      for (int kb = 0; kb < 2; ++kb) {
        const uint64_t da = make_kmajor_sw128_desc(sm0 + kb * (kAttnPairs * 128)), db = make_kmajor_sw128_desc(kst + kb * (kAtKeys * 128));
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4) tc_mma(tmem_base + b * kAtKeys, da + 2 * k4, db + 2 * k4, idesc_s, (kb | k4) != 0);
      }
      tc_commit(smem_u32(k_empty + st));
      tc_commit(smem_u32(s_full + b));
    };
    if (n_tiles > 0) issue_s(0);
    for (int i = 0; i < n_tiles && ok; ++i) {
      if (i + 1 < n_tiles) {
        issue_s(i + 1);
        if (!ok) break;
      }
      if (!(ok = mbar_wait_warp(smem_u32(p_full), i & 1, abort_flag, status, 55))) break;
      if (!(ok = mbar_wait_warp(smem_u32(vt_full + (i & 1)), (i >> 1) & 1, abort_flag, status, 56))) break;
      tc_fence_after();
      const uint64_t db = make_kmajor_sw128_desc(sm0 + kAtOffVt + (i & 1) * kAtVtBytes);
#pragma unroll
      for (int h = 0; h < 2; ++h) {                          // P hi, then P lo
        const uint64_t da = make_kmajor_sw128_desc(sm0 + kAtOffP + h * (kAttnPairs * 128));
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4) tc_mma(tm_o, da + 2 * k4, db + 2 * k4, idesc_o, (i | h | k4) != 0);
      }
      tc_commit(smem_u32(vt_empty + (i & 1)));
      tc_commit(smem_u32(pv_done));
    }
  } else {
    // ------------------------------ softmax ------------------------------
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;       // this warp's quarter of the lanes of tensor memory
    const uint32_t tm_o = tmem_base + lane_base + 2 * kAtKeys;
    const int pr = tid;                                      // pair = lane of tensor memory = row of P
    const float sl2 = rsqrtf((float)kAtD) * 1.4426950408889634f;      // scores in base 2
    bool ok = true;
    for (int i = 0; i < n_tiles && ok; ++i) {
      const int b = i & 1;
      if (!(ok = mbar_wait_warp(smem_u32(s_full + b), (i >> 1) & 1, abort_flag, status, 57))) break;
      tc_fence_after();
      float sc[kAtKeys];
      {
        const uint32_t tm_s = tmem_base + lane_base + b * kAtKeys;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          uint32_t r0[8], r1[8], r2[8], r3[8];
          tmem_ld8_issue(tm_s + half * 32, r0);
          tmem_ld8_issue(tm_s + half * 32 + 8, r1);
          tmem_ld8_issue(tm_s + half * 32 + 16, r2);
          tmem_ld8_issue(tm_s + half * 32 + 24, r3);
          tmem_ld_wait(r0, r1, r2, r3);
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            sc[half * 32 + e] = __uint_as_float(r0[e]);
            sc[half * 32 + 8 + e] = __uint_as_float(r1[e]);
            sc[half * 32 + 16 + e] = __uint_as_float(r2[e]);
            sc[half * 32 + 24 + e] = __uint_as_float(r3[e]);
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(s_empty + b));      // the tensor core may write the scores of tile i + 2 here
      // scale, mask the keys past the end (last tile only), the tile's maximum
      const int key0 = (t_begin + i) * kAtKeys;
      const bool ragged = key0 + kAtKeys > n_keys;
      float mx = kNegInf;
#pragma unroll
      for (int e = 0; e < kAtKeys; ++e) {
        if (ragged && key0 + e >= n_keys) sc[e] = kNegInf;
        mx = fmaxf(mx, sc[e]);
      }
      mx *= sl2;                                             // sl2 > 0: the maximum of the scaled scores
      // the maximum in use moves only when it has to: P stays below 2^8, far inside fp32 and the bf16 pair
      const bool move = mx > m_used + kAtRescale;            // always on the first tile (m_used = -inf)
      float corr = 1.f;
      if (move) {
        corr = at_ex2(m_used - mx);                          // 0 on the first tile
        m_used = mx;
        l_run *= corr;
      }
      float sum = 0.f;
      const float neg_m = -m_used;
#pragma unroll
      for (int e = 0; e < kAtKeys; ++e) {
        sc[e] = at_ex2(fmaf(sc[e], sl2, neg_m));             // scale and shift in one operation
        sum += sc[e];
      }
      l_run += sum;
      // O and P belong to the tensor core until P V of the previous tile is complete
      if (i > 0) {
        if (!(ok = mbar_wait_warp(smem_u32(pv_done), (i - 1) & 1, abort_flag, status, 58))) break;
        tc_fence_after();
        if (__any_sync(0xffffffffu, move)) {
#pragma unroll 1
          for (int c0 = 0; c0 < kAtD; c0 += 32) {
            uint32_t r0[8], r1[8], r2[8], r3[8];
            tmem_ld8_issue(tm_o + c0, r0);
            tmem_ld8_issue(tm_o + c0 + 8, r1);
            tmem_ld8_issue(tm_o + c0 + 16, r2);
            tmem_ld8_issue(tm_o + c0 + 24, r3);
            tmem_ld_wait(r0, r1, r2, r3);
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              r0[e] = __float_as_uint(__uint_as_float(r0[e]) * corr);
              r1[e] = __float_as_uint(__uint_as_float(r1[e]) * corr);
              r2[e] = __float_as_uint(__uint_as_float(r2[e]) * corr);
              r3[e] = __float_as_uint(__uint_as_float(r3[e]) * corr);
            }
            tmem_st8(tm_o + c0, r0);
            tmem_st8(tm_o + c0 + 8, r1);
            tmem_st8(tm_o + c0 + 16, r2);
            tmem_st8(tm_o + c0 + 24, r3);
          }
          tmem_st_wait();
        }
      }
      // P as hi + lo: row pr of two [128 rows][128 B] tiles, 8 keys per 16-byte piece
      unsigned char* prow = smem + kAtOffP;
#pragma unroll
      for (int c = 0; c < kAtKeys / 8; ++c) {
        uint4 hi, lo;
        at_split2(sc[c * 8 + 0], sc[c * 8 + 1], hi.x, lo.x);
        at_split2(sc[c * 8 + 2], sc[c * 8 + 3], hi.y, lo.y);
        at_split2(sc[c * 8 + 4], sc[c * 8 + 5], hi.z, lo.z);
        at_split2(sc[c * 8 + 6], sc[c * 8 + 7], hi.w, lo.w);
        const uint32_t off = sw128(pr, c);
        *reinterpret_cast<uint4*>(prow + off) = hi;
        *reinterpret_cast<uint4*>(prow + kAttnPairs * 128 + off) = lo;
      }
      fence_async_smem();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(p_full));
    }
    // ---- the CTA's partial result: (maximum, sum, unnormalised output) of its pairs into shared memory ----
    if (ok && n_tiles > 0) ok = mbar_wait_warp(smem_u32(pv_done), (n_tiles - 1) & 1, abort_flag, status, 59);
    tc_fence_after();
    float* s_o = reinterpret_cast<float*>(smem + kAtOffK);     // [128][kAtOStride]: the key / value stages are idle now
    const bool have = ok && n_tiles > 0;
    s_m[pr] = have ? m_used : kNegInf;
    s_l[pr] = have ? l_run : 0.f;
#pragma unroll 1
    for (int c0 = 0; c0 < kAtD; c0 += 32) {
      uint32_t r0[8], r1[8], r2[8], r3[8];
      if (have) {                                            // warp-uniform
        tmem_ld8_issue(tm_o + c0, r0);
        tmem_ld8_issue(tm_o + c0 + 8, r1);
        tmem_ld8_issue(tm_o + c0 + 16, r2);
        tmem_ld8_issue(tm_o + c0 + 24, r3);
        tmem_ld_wait(r0, r1, r2, r3);
      } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) r0[e] = r1[e] = r2[e] = r3[e] = 0u;
      }
      float4* dst = reinterpret_cast<float4*>(s_o + (size_t)pr * kAtOStride + c0);
      dst[0] = make_float4(__uint_as_float(r0[0]), __uint_as_float(r0[1]), __uint_as_float(r0[2]), __uint_as_float(r0[3]));
      dst[1] = make_float4(__uint_as_float(r0[4]), __uint_as_float(r0[5]), __uint_as_float(r0[6]), __uint_as_float(r0[7]));
      dst[2] = make_float4(__uint_as_float(r1[0]), __uint_as_float(r1[1]), __uint_as_float(r1[2]), __uint_as_float(r1[3]));
      dst[3] = make_float4(__uint_as_float(r1[4]), __uint_as_float(r1[5]), __uint_as_float(r1[6]), __uint_as_float(r1[7]));
      dst[4] = make_float4(__uint_as_float(r2[0]), __uint_as_float(r2[1]), __uint_as_float(r2[2]), __uint_as_float(r2[3]));
      dst[5] = make_float4(__uint_as_float(r2[4]), __uint_as_float(r2[5]), __uint_as_float(r2[6]), __uint_as_float(r2[7]));
      dst[6] = make_float4(__uint_as_float(r3[0]), __uint_as_float(r3[1]), __uint_as_float(r3[2]), __uint_as_float(r3[3]));
      dst[7] = make_float4(__uint_as_float(r3[4]), __uint_as_float(r3[5]), __uint_as_float(r3[6]), __uint_as_float(r3[7]));
    }
  }

  // ------------------------------ merge over the cluster, teardown ------------------------------
  tc_fence_before();
  __syncthreads();
  cg::cluster_group cluster = cg::this_cluster();
  cluster.sync();
  if (tid < 256 && !*abort_flag) {
    // rank z merges rows z * R .. z * R + R - 1 of all partials (distributed shared memory) and writes them
    float* s_o = reinterpret_cast<float*>(smem + kAtOffK);
    constexpr int TPR = kAtD / 4;                           // threads per row (one float4 each)
    const int R = kAttnPairs / n_splits;
    const int c4 = tid % TPR;
    for (int i = tid / TPR; i < R; i += 256 / TPR) {
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
        const float f = at_ex2(mk[k] - mx);                  // 0 for a split without keys (its maximum is -inf)
        den = fmaf(f, *cluster.map_shared_rank(&s_l[pr], k), den);
        const float4 v = *reinterpret_cast<const float4*>(cluster.map_shared_rank(s_o + (size_t)pr * kAtOStride + c4 * 4, k));
        acc.x = fmaf(f, v.x, acc.x); acc.y = fmaf(f, v.y, acc.y); acc.z = fmaf(f, v.z, acc.z); acc.w = fmaf(f, v.w, acc.w);
      }
      const int cr = gp / rep, j = gp - cr * rep;
      float* dst = a.out + ((size_t)(row0 + s_list[cr]) * a.Hq + g * rep + j) * kAtD + c4 * 4;
      const float inv = 1.f / den;
      *reinterpret_cast<float4*>(dst) = make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
    }
  }
  cluster.sync();                                          // peers may still be reading this CTA's partial
  if (warp == 4) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kAtTmemCols) : "memory");
  }
}

cudaError_t configure_attention_tc() {
  static std::mutex mu;
  static bool done[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  std::lock_guard<std::mutex> lock(mu);
  if (dev >= 0 && dev < 64 && done[dev]) return cudaSuccess;
  e = cudaFuncSetAttribute(k_block_attention_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, kAtSmemBytes);
  if (e == cudaSuccess && dev >= 0 && dev < 64) done[dev] = true;
  return e;
}

cudaError_t launch_attention_tc(const AttnArgs& a, int m_tiles, int n_splits, cudaStream_t s) {
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(m_tiles, a.S * a.B * a.Hkv, n_splits);
  lc.blockDim = dim3(kAtThreads);
  lc.dynamicSmemBytes = kAtSmemBytes;
  lc.stream = s;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = 1; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = n_splits;
  lc.attrs = at;
  lc.numAttrs = 1;
  return cudaLaunchKernelEx(&lc, k_block_attention_tc, a, n_splits);
}

}  // namespace team
