// Grouped SwiGLU expert kernel for bf16 weights on sm_100a: TMA-staged weight tiles, tcgen05.mma
// with accumulators in tensor memory, SwiGLU and the routing-weight scatter-combine fused in.
//
// Work is measured in "groups": 16 consecutive columns of one work item's intermediate dimension
// (a work item is a run of up to NT token-slots of one activated expert, built by the selection
// kernel).  A group costs the same HBM bytes everywhere (16 gate rows + 16 up rows + a 16-column
// strip of W_down), so the global list of groups is cut into one contiguous range per CTA and every
// SM streams the same number of bytes (+- one group).  A CTA walks its range in chunks: the part of
// the range that falls into one 64-column window of one item (1 to 4 groups).  For a chunk it
//   phase 1  streams the chunk's W_gate / W_up rows against the gathered token rows,
//            D1[128, N] = A[128, H] * X[N, H]^T  (weights on M, tokens on N).  One 4-D TMA box per
//            64-wide k-block delivers the rows already interleaved as [group][gate 16 | up 16], so a
//            gate row and its up row sit in the same warp's TMEM lanes.
//   SwiGLU   reads D1 from TMEM, a = silu(gate) * up, writes a as bf16 into shared memory in the
//            K-major 128B-swizzled layout the tensor core reads as a B operand
//   phase 2  streams W_down[e, :, window] in 128-row tiles: D2[128, N] = Wd_tile[128, cols] * a[N, cols]^T
//            over the chunk's columns, multiplies by the slot's routing weight and adds into y[row, h]
//            with fp32 reductions.
// Every weight byte of an activated expert is read from HBM once per step (two CTAs that share a
// window read its W_down tiles at the same time, odd CTAs walking their range backwards, so the
// second read is served by L2); nothing but y is written.
//
// Warp roles (256 threads): warp 0 = TMA producer, warp 1 = MMA issuer + TMEM owner, warp 2 = token
// gather (cp.async into the swizzled B tile), warp 3 idle, warps 4-7 = epilogue (one TMEM lane
// quarter each).  All waits are bounded; on expiry the kernel records TEAM_ERR_TIMEOUT, drains and
// frees its tensor memory.
#include <cuda.h>

#include "team_common.cuh"

namespace team {

constexpr int kTcThreads = 256;
constexpr int kATileBytes = 128 * 128;          // 128 rows x 64 bf16
constexpr int kGroupCols = 16;                  // intermediate columns per group (the unit of balance)
constexpr int kWindowCols = 64;                 // columns per window (one 128-byte swizzle row of W_down)
constexpr unsigned long long kWaitCycles = 2000000000ull;   // ~1 s at 2 GHz

template <int NT>
struct TcCfg {
  static constexpr int kBTileBytes = NT * 128;
  static constexpr int kStageBytes = kATileBytes + kBTileBytes;
  static constexpr int kStages = (NT <= 32) ? 10 : (NT <= 64 ? 8 : 6);
  static constexpr int kActBytes = NT * 128;
  static constexpr int kTmemCols = (3 * NT <= 128) ? 128 : (3 * NT <= 256 ? 256 : 512);
  static constexpr int kBarBytes = (3 * kStages + 8) * 8;
  static constexpr int kTableBytes = 4 * NT * 8 + NT * 4;   // per-epilogue-warp (row, weight) + gather rows
  static constexpr int kSmemBytes = 1024 + kStages * kStageBytes + kActBytes + kBarBytes + kTableBytes + 64;
};

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false when it gave up (or another thread of the CTA already did).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status,
                                          int where) {
  if (mbar_try(bar, parity)) return true;
  const unsigned long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
      if (mbar_try(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > kWaitCycles) {
      *abort_flag = 1;
      set_status(status, TEAM_ERR_TIMEOUT, where);
      return false;
    }
  }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
      : "memory");
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                            uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar)
      : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// D[tmem] (+)= A[smem desc] * B[smem desc]^T, bf16 inputs, fp32 accumulate, M = 128.
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// Shared-memory matrix descriptor: K-major, 128-byte swizzle, rows 128 B apart, 8-row groups 1024 B apart.
__device__ __forceinline__ uint64_t make_kmajor_sw128_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);   // start address, 16-byte units
  d |= (uint64_t)1 << 16;                         // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;               // stride byte offset: 8 rows * 128 B
  d |= (uint64_t)1 << 46;                         // descriptor version for tcgen05
  d |= (uint64_t)2 << 61;                         // layout: 128-byte swizzle
  return d;
}

// Instruction descriptor: D fp32, A and B bf16, both K-major, M = 128, N = n (multiple of 16).
__device__ __forceinline__ uint32_t make_idesc_bf16(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}

__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float (&v)[8]) {
  uint32_t r0, r1, r2, r3, r4, r5, r6, r7;
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3), "=r"(r4), "=r"(r5), "=r"(r6), "=r"(r7)
               : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
  v[0] = __uint_as_float(r0); v[1] = __uint_as_float(r1); v[2] = __uint_as_float(r2); v[3] = __uint_as_float(r3);
  v[4] = __uint_as_float(r4); v[5] = __uint_as_float(r5); v[6] = __uint_as_float(r6); v[7] = __uint_as_float(r7);
}

// ---------------------------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------------------------
struct TcArgs {
  const __nv_bfloat16* x;      // [T, H]
  const int32_t* perm;         // slot ids grouped by expert
  const float* topk_w;         // [T, k]
  const WorkItem* items;
  const int32_t* n_items;
  float* y;                    // [T, H], pre-zeroed rows of computed tokens
  int32_t* status;
  Dims d;
  int gate_first;              // 1: the 4-D box delivers [gate | up] per group, 0: [up | gate]
};

// Tensor maps: gu[g-1] = W_gate/W_up viewed as {H, 16 rows, 2 (gate, up), rows/16} with a box of g
// groups; down = W_down as {I, rows} with a [128 x 64] box.
struct TcMaps {
  CUtensorMap gu[4];
  CUtensorMap down;
};

// One step of a CTA's walk over its group range.
struct Chunk {
  int item;     // work item
  int window;   // 64-column window of the intermediate dimension
  int g0;       // first group of the window that belongs to the chunk (0..3)
  int g;        // groups in the chunk (1..4)
};

struct ChunkWalker {
  long long lo, hi, cur;
  int NG;
  bool reverse;
  __device__ ChunkWalker(long long lo_, long long hi_, int ng, bool rev)
      : lo(lo_), hi(hi_), cur(rev ? hi_ : lo_), NG(ng), reverse(rev) {}
  __device__ bool next(Chunk& c) {
    if (!reverse) {
      if (cur >= hi) return false;
      const long long item = cur / NG;
      const int j = (int)(cur - item * NG);
      long long end = item * NG + (j / 4 + 1) * 4;
      if (end > hi) end = hi;
      c.item = (int)item; c.window = j / 4; c.g0 = j % 4; c.g = (int)(end - cur);
      cur = end;
    } else {
      if (cur <= lo) return false;
      const long long last = cur - 1, item = last / NG;
      const int j = (int)(last - item * NG);
      long long begin = item * NG + (j / 4) * 4;
      if (begin < lo) begin = lo;
      c.item = (int)item; c.window = j / 4; c.g0 = (int)(begin - item * NG) % 4; c.g = (int)(cur - begin);
      cur = begin;
    }
    return true;
  }
};

template <int NT>
__global__ void __launch_bounds__(kTcThreads, 1)
k_experts_tc(const __grid_constant__ TcMaps maps, TcArgs a) {
  using C = TcCfg<NT>;
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  unsigned char* act_tile = smem + C::kStages * C::kStageBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(act_tile + C::kActBytes);
  uint64_t* bar_fullA = bars;
  uint64_t* bar_fullB = bars + C::kStages;
  uint64_t* bar_empty = bars + 2 * C::kStages;
  uint64_t* bar_misc = bars + 3 * C::kStages;   // 0 acc1_full, 1 acc1_empty, 2 act_ready, 3-4 acc2_full, 5-6 acc2_empty
  int32_t* tbl_row = reinterpret_cast<int32_t*>(reinterpret_cast<unsigned char*>(bars) + C::kBarBytes);   // [4][NT]
  float* tbl_wt = reinterpret_cast<float*>(tbl_row + 4 * NT);                                             // [4][NT]
  int32_t* gather_row = reinterpret_cast<int32_t*>(tbl_wt + 4 * NT);                                      // [NT]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gather_row + NT);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const Dims d = a.d;
  const int KB = d.H / 64;          // k-blocks of phase 1
  const int HT = d.H / 128;         // row tiles of phase 2
  const int NG = d.I / kGroupCols;  // groups per work item

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::kStages; ++s) {
      mbar_init(smem_u32(bar_fullA + s), 1);
      mbar_init(smem_u32(bar_fullB + s), 32);
      mbar_init(smem_u32(bar_empty + s), 1);
    }
    mbar_init(smem_u32(bar_misc + 0), 1);
    mbar_init(smem_u32(bar_misc + 1), 128);
    mbar_init(smem_u32(bar_misc + 2), 128);
    mbar_init(smem_u32(bar_misc + 3), 1);
    mbar_init(smem_u32(bar_misc + 4), 1);
    mbar_init(smem_u32(bar_misc + 5), 128);
    mbar_init(smem_u32(bar_misc + 6), 128);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"((uint32_t)C::kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_acc1 = tmem_base;

  // This CTA's contiguous range of groups; odd CTAs walk it backwards so that the two CTAs sharing a
  // window touch its W_down tiles at the same time.
  const long long n_groups = (long long)(*a.n_items) * NG;
  const long long g_lo = n_groups * blockIdx.x / gridDim.x, g_hi = n_groups * (blockIdx.x + 1) / gridDim.x;
  const bool reverse = (blockIdx.x & 1) != 0;

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      ChunkWalker walk(g_lo, g_hi, NG, reverse);
      Chunk c;
      while (ok && walk.next(c)) {
        const WorkItem item = a.items[c.item];
        const int col0 = c.window * kWindowCols + c.g0 * kGroupCols;
        const int grp = (item.e * d.I + col0) / kGroupCols;          // coordinate in units of 16 rows
        const CUtensorMap* gu = &maps.gu[c.g - 1];
        const uint32_t bytes1 = (uint32_t)c.g * 4096u;
        for (int kb = 0; kb < KB; ++kb, ++it) {
          const uint32_t s = it % C::kStages, par = (it / C::kStages) & 1;
          if (!(ok = mbar_wait(smem_u32(bar_empty + s), par ^ 1, abort_flag, a.status, 1))) break;
          const uint32_t dst = smem_u32(smem + s * C::kStageBytes), bar = smem_u32(bar_fullA + s);
          mbar_arrive_expect_tx(bar, bytes1);
          tma_load_4d(dst, gu, kb * 64, 0, 0, grp, bar);
        }
        if (!ok) break;
        for (int ht = 0; ht < HT; ++ht, ++it) {
          const uint32_t s = it % C::kStages, par = (it / C::kStages) & 1;
          if (!(ok = mbar_wait(smem_u32(bar_empty + s), par ^ 1, abort_flag, a.status, 2))) break;
          const uint32_t dst = smem_u32(smem + s * C::kStageBytes), bar = smem_u32(bar_fullA + s);
          mbar_arrive_expect_tx(bar, kATileBytes);
          tma_load_2d(dst, &maps.down, c.window * kWindowCols, item.e * d.H + ht * 128, bar);
        }
      }
      if (*abort_flag) {
        // Let copies already in flight land before the CTA's shared memory is released.
        const uint32_t back = it < (uint32_t)C::kStages ? it : (uint32_t)C::kStages;
        for (uint32_t j = it - back; j < it; ++j) {
          const uint32_t s = j % C::kStages, par = (j / C::kStages) & 1;
          const unsigned long long t0 = clock64();
          while (!mbar_try(smem_u32(bar_fullA + s), par) && clock64() - t0 < kWaitCycles / 16) {}
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    if (lane == 0) {
      uint32_t it = 0, chunk_i = 0, t2 = 0, bphase = 0;
      bool ok = true;
      const uint64_t act_desc = make_kmajor_sw128_desc(smem_u32(act_tile));
      ChunkWalker walk(g_lo, g_hi, NG, reverse);
      Chunk c;
      for (; ok && walk.next(c); ++chunk_i) {
        const WorkItem item = a.items[c.item];
        const int N = (item.n + 15) & ~15;
        const uint32_t idesc = make_idesc_bf16(N);
        if (!(ok = mbar_wait(smem_u32(bar_misc + 1), (chunk_i & 1) ^ 1, abort_flag, a.status, 3))) break;
        tc_fence_after();
        for (int kb = 0; kb < KB; ++kb, ++it) {
          const uint32_t s = it % C::kStages, par = (it / C::kStages) & 1;
          if (!(ok = mbar_wait(smem_u32(bar_fullA + s), par, abort_flag, a.status, 4))) break;
          if (!(ok = mbar_wait(smem_u32(bar_fullB + s), (bphase >> s) & 1, abort_flag, a.status, 5))) break;
          bphase ^= 1u << s;
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + s * C::kStageBytes);
          const uint64_t da = make_kmajor_sw128_desc(sa), db = make_kmajor_sw128_desc(sa + kATileBytes);
#pragma unroll
          for (int k4 = 0; k4 < 4; ++k4)
            tc_mma(tmem_acc1, da + 2 * k4, db + 2 * k4, idesc, (kb | k4) != 0);
          tc_commit(smem_u32(bar_empty + s));
        }
        if (!ok) break;
        tc_commit(smem_u32(bar_misc + 0));
        if (!(ok = mbar_wait(smem_u32(bar_misc + 2), chunk_i & 1, abort_flag, a.status, 6))) break;
        tc_fence_after();
        for (int ht = 0; ht < HT; ++ht, ++it, ++t2) {
          const uint32_t b = t2 & 1, u = t2 >> 1;
          if (!(ok = mbar_wait(smem_u32(bar_misc + 5 + b), (u & 1) ^ 1, abort_flag, a.status, 7))) break;
          const uint32_t s = it % C::kStages, par = (it / C::kStages) & 1;
          if (!(ok = mbar_wait(smem_u32(bar_fullA + s), par, abort_flag, a.status, 8))) break;
          tc_fence_after();
          const uint64_t da = make_kmajor_sw128_desc(smem_u32(smem + s * C::kStageBytes));
          const uint32_t acc2 = tmem_base + NT * (1 + b);
          // the chunk's columns are k-steps g0 .. g0+g-1 of the window tile and 0 .. g-1 of the activation tile
          for (int kk = 0; kk < c.g; ++kk) tc_mma(acc2, da + 2 * (c.g0 + kk), act_desc + 2 * kk, idesc, kk != 0);
          tc_commit(smem_u32(bar_empty + s));
          tc_commit(smem_u32(bar_misc + 3 + b));
        }
      }
    }
    __syncwarp();
  } else if (warp == 2) {
    // ------------------------------ token gather (B operand of phase 1) ------------------------------
    constexpr int kLag = 3;   // stages of cp.async kept in flight
    uint32_t it = 0;
    bool ok = true;
    ChunkWalker walk(g_lo, g_hi, NG, reverse);
    Chunk c;
    while (ok && walk.next(c)) {
      const WorkItem item = a.items[c.item];
      for (int r = lane; r < item.n; r += 32) {
        int row;
        float wt;
        slot_row_weight(a.perm[item.begin + r], d.T, d.k, a.topk_w, row, wt);
        gather_row[r] = row;
      }
      __syncwarp();
      const int chunks = item.n * 8;
      int pending = 0;
      for (int kb = 0; kb < KB; ++kb, ++it) {
        const uint32_t s = it % C::kStages, par = (it / C::kStages) & 1;
        ok = mbar_wait(smem_u32(bar_empty + s), par ^ 1, abort_flag, a.status, 9);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        const uint32_t dstB = smem_u32(smem + s * C::kStageBytes + kATileBytes);
        for (int ch16 = lane; ch16 < chunks; ch16 += 32) {
          const int r = ch16 >> 3, ch = ch16 & 7;
          const __nv_bfloat16* src = a.x + (size_t)gather_row[r] * d.H + kb * 64 + ch * 8;
          const uint32_t dst = dstB + r * 128 + ((ch ^ (r & 7)) << 4);
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        if (++pending > kLag) {
          asm volatile("cp.async.wait_group %0;" ::"n"(kLag) : "memory");
          fence_async_smem();
          mbar_arrive(smem_u32(bar_fullB + (it - kLag) % C::kStages));
          --pending;
        }
      }
      asm volatile("cp.async.wait_group 0;" ::: "memory");
      fence_async_smem();
      if (ok)
        for (int j = pending; j > 0; --j) mbar_arrive(smem_u32(bar_fullB + (it - j) % C::kStages));
      __syncwarp();
      // Phase-2 stages carry no B tile, but the ring's empty barriers must still be observed one
      // round at a time: a parity wait that skipped a round could be satisfied by an older phase.
      for (int ht = 0; ok && ht < HT; ++ht, ++it) {
        const uint32_t s = it % C::kStages, par = (it / C::kStages) & 1;
        ok = mbar_wait(smem_u32(bar_empty + s), par ^ 1, abort_flag, a.status, 12);
        ok = __all_sync(0xffffffffu, ok);
      }
    }
  } else if (warp >= 4) {
    // ------------------------------ epilogue ------------------------------
    const int q = warp - 4;                       // TMEM lane quarter == warp_id % 4 == group inside the chunk
    int32_t* my_row = tbl_row + q * NT;
    float* my_wt = tbl_wt + q * NT;
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    uint32_t chunk_i = 0, t2 = 0;
    bool ok = true;
    ChunkWalker walk(g_lo, g_hi, NG, reverse);
    Chunk c;
    for (; ok && walk.next(c); ++chunk_i) {
      const WorkItem item = a.items[c.item];
      const int N = (item.n + 15) & ~15;
      __syncwarp();
      for (int r = lane; r < item.n; r += 32) {
        int row;
        float wt;
        slot_row_weight(a.perm[item.begin + r], d.T, d.k, a.topk_w, row, wt);
        my_row[r] = row;
        my_wt[r] = wt;
      }
      __syncwarp();
      // ---- SwiGLU: TMEM -> registers -> bf16 activation tile (B operand of phase 2) ----
      ok = mbar_wait(smem_u32(bar_misc + 0), chunk_i & 1, abort_flag, a.status, 10);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      if (q < c.g) {
        const int i_local = q * 16 + (lane & 15);     // column of the activation tile this lane pair owns
        const bool first_half = lane < 16;
        for (int c0 = 0; c0 < N; c0 += 8) {
          float v[8];
          tmem_ld8(tmem_acc1 + lane_off + c0, v);
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float o = __shfl_xor_sync(0xffffffffu, v[j], 16);
            const bool mine_is_gate = (first_half == (a.gate_first != 0));
            const float g = mine_is_gate ? v[j] : o;
            const float u = mine_is_gate ? o : v[j];
            v[j] = g / (1.f + expf(-g)) * u;
          }
          // lanes 0-15 store columns c0..c0+3, lanes 16-31 store c0+4..c0+7
          const int jb = first_half ? 0 : 4;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int n = c0 + jb + j;
            const uint32_t off = n * 128 + (((i_local >> 3) ^ (n & 7)) << 4) + (i_local & 7) * 2;
            *reinterpret_cast<__nv_bfloat16*>(act_tile + off) = __float2bfloat16_rn(v[jb + j]);
          }
        }
      }
      tc_fence_before();
      mbar_arrive(smem_u32(bar_misc + 1));
      fence_async_smem();
      mbar_arrive(smem_u32(bar_misc + 2));
      // ---- down projection tiles: scale by routing weight, add into y ----
      for (int ht = 0; ht < HT; ++ht, ++t2) {
        const uint32_t b = t2 & 1, u = t2 >> 1;
        ok = mbar_wait(smem_u32(bar_misc + 3 + b), u & 1, abort_flag, a.status, 11);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        const uint32_t acc2 = tmem_base + NT * (1 + b) + lane_off;
        float* ycol = a.y + ht * 128 + q * 32 + lane;
        for (int c0 = 0; c0 < N; c0 += 8) {
          float v[8];
          tmem_ld8(acc2 + c0, v);
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const int n = c0 + j;
            if (n < item.n) atomicAdd(ycol + (size_t)my_row[n] * d.H, my_wt[n] * v[j]);
          }
        }
        tc_fence_before();
        mbar_arrive(smem_u32(bar_misc + 5 + b));
      }
    }
  }

  // ------------------------------ teardown ------------------------------
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)C::kTmemCols)
                 : "memory");
  }
}

// ---------------------------------------------------------------------------------------------
// Host side: tensor maps and launch
// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

size_t experts_tc_maps_bytes() { return sizeof(TcMaps); }

// Builds the five tensor maps for a layer.  w_gate / w_up: bf16 [rows_gu, H]; w_down: bf16 [rows_d, I].
// Returns 0, or a driver error code / -1.  *gate_first tells the kernel which of gate / up comes
// first inside a group (the 4-D view needs a positive stride between the two matrices).
int make_expert_maps(void* out_maps, const void* w_gate, const void* w_up, const void* w_down, uint64_t rows_gu,
                     uint64_t H, uint64_t rows_d, uint64_t I, int* gate_first) {
  EncodeTiledFn fn = get_encode_fn();
  if (fn == nullptr) return -1;
  TcMaps* m = reinterpret_cast<TcMaps*>(out_maps);
  const uintptr_t pg = reinterpret_cast<uintptr_t>(w_gate), pu = reinterpret_cast<uintptr_t>(w_up);
  *gate_first = pu > pg ? 1 : 0;
  const uintptr_t base = pu > pg ? pg : pu, delta = pu > pg ? pu - pg : pg - pu;
  if (delta == 0 || (delta & 15) || delta >= (1ull << 40)) return -2;
  for (int g = 1; g <= 4; ++g) {
    cuuint64_t dims[4] = {H, 16, 2, rows_gu / 16};
    cuuint64_t strides[3] = {H * 2, delta, 16 * H * 2};
    cuuint32_t box[4] = {64, 16, 2, (cuuint32_t)g};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = fn(&m->gu[g - 1], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, reinterpret_cast<void*>(base), dims, strides,
                    box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return (int)r;
  }
  cuuint64_t dims[2] = {I, rows_d};
  cuuint64_t strides[1] = {I * 2};
  cuuint32_t box[2] = {64, 128};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(&m->down, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(w_down), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : (int)r;
}

template <int NT>
static cudaError_t launch_tc(const void* maps, TcArgs args, int grid, cudaStream_t s) {
  using C = TcCfg<NT>;
  k_experts_tc<NT><<<grid, kTcThreads, C::kSmemBytes, s>>>(*reinterpret_cast<const TcMaps*>(maps), args);
  return cudaGetLastError();
}

cudaError_t configure_experts_tc(int item_tile) {
  switch (item_tile) {
    case 32: return cudaFuncSetAttribute(k_experts_tc<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, TcCfg<32>::kSmemBytes);
    case 64: return cudaFuncSetAttribute(k_experts_tc<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, TcCfg<64>::kSmemBytes);
    case 128: return cudaFuncSetAttribute(k_experts_tc<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, TcCfg<128>::kSmemBytes);
    default: return cudaErrorInvalidValue;
  }
}

cudaError_t launch_experts_tc(const void* maps, int gate_first, int item_tile, const void* x, Workspace ws, float* y,
                              Dims d, int grid, cudaStream_t s) {
  TcArgs a;
  a.x = static_cast<const __nv_bfloat16*>(x);
  a.perm = ws.r.perm;
  a.topk_w = ws.r.topk_w;
  a.items = ws.items;
  a.n_items = ws.n_items;
  a.y = y;
  a.status = ws.status;
  a.d = d;
  a.gate_first = gate_first;
  switch (item_tile) {
    case 32: return launch_tc<32>(maps, a, grid, s);
    case 64: return launch_tc<64>(maps, a, grid, s);
    case 128: return launch_tc<128>(maps, a, grid, s);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace team
