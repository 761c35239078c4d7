// Grouped SwiGLU expert kernel for bf16 weights on sm_100a: weight tiles streamed into a shared-memory
// ring, tcgen05.mma with accumulators in tensor memory, SwiGLU and the routing-weight
// scatter-combine fused in.
//
// Unit of work and balance.  A work item is a run of up to NT token-slots of one activated expert
// (built by the selection kernel).  Its intermediate dimension is cut into "groups" of 16 columns.
// A group costs the same HBM bytes everywhere:
//     phase 1   16 rows of W_gate + 16 rows of W_up (full hidden width), and
//     phase 2   a quarter of the W_down tiles of the group's 64-column "window": the g-th group of
//               a window owns the hidden-row tiles [g*HT/4, (g+1)*HT/4) of that window,
// so the global list of groups is cut into one contiguous range per CTA and every SM streams the
// same number of bytes (+- one group) and every weight byte of an activated expert is requested
// exactly once per step.
//
// A CTA walks its range in super-chunks of up to kScWindows windows (of any items):
//   phase 1   D1[128, N] = A[128, H] * X[N, H]^T per tile of up to 4 consecutive groups (weights on M,
//             tokens on N); tile rows are ordered [group][gate 16 | up 16], so a gate row and its up
//             row sit in the same warp's TMEM lanes.
//   SwiGLU    a = silu(gate) * up from TMEM, rounded to bf16 and published to a small global
//             scratch [item][token][I]; a per-window counter says how many of its 4 groups are there.
//   phase 2   for each of its groups' W_down tiles: D2[128, N] = Wd[128, 64] * a[N, 64]^T over the
//             whole window (the window's activations are read back from the scratch once all four
//             groups are published, whichever CTAs computed them), times the slot's routing weight,
//             added into y[row, h] with fp32 reductions.
// A window cut by a range boundary is shared by neighbouring CTAs.  Its phase-2 tiles wait for the
// neighbours' activations; the tiles of a CTA's first (head) window are therefore done last.  No
// publish ever waits on another CTA, so the waits cannot form a cycle; the launch is cooperative so
// that all CTAs are resident, and every wait is bounded.
//
// Loads.  Eight loader warps fill the ring with cp.async: every warp instruction fetches kKbs * 128
// contiguous bytes of one weight row (phase 1) or 128-byte row pieces of four rows (phase 2) and
// scatters them into the K-major, 128-byte-swizzled tiles the tensor core reads; the stage's
// mbarrier is armed to fire when the copies land (cp.async.mbarrier.arrive), so a loader only ever
// blocks on a free slot.  (Measured on B200: tiled TMA boxes deliver 128-byte pieces of
// 4 KB-strided rows at 3.6-5.7 TB/s; these requests reach 7 TB/s.)  A stage holds kKbs consecutive
// k-blocks of the tile (or kKbs W_down tiles) plus the matching slices of the token rows.
// Two operand modes:
//   resident-N (T <= 16 rows, N = 16): every expert is applied to all rows of x; rows not routed
//              to the expert get weight 0 in the combine.
//   gather     (N = 16..NT): the loaders gather the item's token rows.
//
// Warp roles (512 threads): warps 0-7 = loaders, warp 8 = MMA issuer + TMEM owner (converged warp,
// one elected lane issues), warp 9 = activation-window loader, warps 12-15 = epilogue (one TMEM lane
// quarter each).  On a wait's expiry the kernel records TEAM_ERR_TIMEOUT, drains and frees its
// tensor memory.
#include "team_common.cuh"

namespace team {

constexpr int kTcThreads = 512;
constexpr int kLoaders = 8;                     // warps 0..7
constexpr int kMmaWarp = 8;
constexpr int kActWarp = 9;
constexpr int kEpiWarp0 = 12;                   // warps 12..15 (warp % 4 = TMEM lane quarter)
constexpr int kATileBytes = 128 * 128;          // 128 rows x 64 bf16
constexpr int kGroupCols = 16;                  // intermediate columns per group (the unit of balance)
constexpr int kWindowCols = 64;                 // columns per window (one 128-byte swizzle row of W_down)
constexpr int kResidentRows = 16;               // N of the resident-N mode
constexpr int kRingBars = 16;                   // stages in flight at most (full / empty barrier pairs)
constexpr int kMaxSmemBytes = 232448;           // dynamic shared memory a CTA may opt in to on sm_100
constexpr unsigned long long kWaitCycles = 2000000000ull;   // ~1 s at 2 GHz

template <int NT>
struct TcCfg {
  static constexpr bool kRes = NT == kResidentRows;
  static constexpr int kKbs = kRes ? 4 : 2;                     // k-blocks (or W_down tiles) per stage
  static constexpr int kABytes = kKbs * kATileBytes;
  static constexpr int kBSub = NT * 128;                        // token tile of one k-block
  static constexpr int kStageBytes = kABytes + kKbs * kBSub;    // a full (4-group) tile's stage
  static constexpr int kActBufs = NT <= 64 ? 2 : 1;             // activation windows staged in shared memory
  static constexpr int kActBytes = NT * 128;                    // NT tokens x 64 columns bf16
  static constexpr int kScWindows = NT <= 16 ? 4 : (NT <= 32 ? 3 : 2);   // windows per super-chunk = phase-1 accumulators
  static constexpr int kAcc2 = NT <= 16 ? 8 : (NT <= 32 ? 4 : 2);
  static constexpr int kTmemUsed = (kScWindows + kAcc2) * NT;
  static constexpr int kTmemCols = kTmemUsed <= 128 ? 128 : (kTmemUsed <= 256 ? 256 : 512);
  static constexpr int kNumBars = 2 * kRingBars + kScWindows + 1 + 2 * kActBufs + 2 * kAcc2;
  static constexpr int kBarBytes = ((kNumBars * 8 + 15) / 16) * 16;
  static constexpr int kTableBytes = 4 * NT * 8 + kLoaders * NT * 4 + kLoaders * kRingBars * 16;   // epilogue (row, weight), loader rows, loader stage queues
  static constexpr int kOtherBytes = 1024 + kActBufs * kActBytes + kBarBytes + kTableBytes + 64;
  static constexpr int kRingBytes = ((kMaxSmemBytes - kOtherBytes) / 1024) * 1024;   // everything that is left
  static constexpr int kSmemBytes = kOtherBytes + kRingBytes;
  static_assert(kRingBytes >= 3 * kStageBytes, "the ring must hold three full-tile stages");
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
// Bounded wait.  Returns false when it gave up (or another thread of the CTA already did).  Every role
// but the MMA issuer backs off between polls (kSleepNs): spinning warps take issue slots from the
// warp that feeds the tensor core.
template <int kSleepNs = 0>
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status,
                                          int where) {
  if (mbar_try(bar, parity)) return true;
  const unsigned long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i) {
      if (mbar_try(bar, parity)) return true;
      if (kSleepNs > 0) __nanosleep(kSleepNs);
    }
    if (*abort_flag) return false;
    if (clock64() - t0 > kWaitCycles) {
      *abort_flag = 1;
      set_status(status, TEAM_ERR_TIMEOUT, where);
      return false;
    }
  }
}
// The same for a whole converged warp: every lane returns the same answer.
template <int kSleepNs = 0>
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status,
                                               int where) {
  return __all_sync(0xffffffffu, mbar_wait<kSleepNs>(bar, parity, abort_flag, status, where));
}

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
// Weight copies: read once per step, so marked evict-first in L2 (the step's small kernels keep their
// working set there: router weights, tables, code).
__device__ __forceinline__ uint64_t stream_policy() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void cp_async16_stream(uint32_t dst, const void* src, uint64_t pol) {
  asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "l"(pol) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
// The barrier receives one arrival from this thread once all of its earlier cp.async copies have landed.
__device__ __forceinline__ void cp_async_arrive(uint32_t bar) {
  asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Issued by a converged warp; one elected lane executes the instruction.  (Measured: issuing from a
// lane inside divergent code costs ~140 cycles per tcgen05.mma, ~50 this way.)
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile(
      "{\n\t.reg .pred q;\n\t"
      "elect.sync _|q, 0xffffffff;\n\t"
      "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
      ::"r"(bar)
      : "memory");
}

// D[tmem] (+)= A[smem desc] * B[smem desc]^T, bf16 inputs, fp32 accumulate, M = 128.
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "elect.sync _|q, 0xffffffff;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
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

// The same load without the wait: the registers are valid only after tmem_ld_wait on them.
__device__ __forceinline__ void tmem_ld8_issue(uint32_t taddr, uint32_t (&r)[8]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr));
}
// Waits for all tensor-memory loads of this thread; the operands tie the loaded registers to the wait.
__device__ __forceinline__ void tmem_ld_wait(uint32_t (&a)[8], uint32_t (&b)[8], uint32_t (&c)[8], uint32_t (&d)[8]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(a[0]), "+r"(a[1]), "+r"(a[2]), "+r"(a[3]), "+r"(a[4]), "+r"(a[5]), "+r"(a[6]), "+r"(a[7]),
                 "+r"(b[0]), "+r"(b[1]), "+r"(b[2]), "+r"(b[3]), "+r"(b[4]), "+r"(b[5]), "+r"(b[6]), "+r"(b[7]),
                 "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3]), "+r"(c[4]), "+r"(c[5]), "+r"(c[6]), "+r"(c[7]),
                 "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3]), "+r"(d[4]), "+r"(d[5]), "+r"(d[6]), "+r"(d[7])
               :
               : "memory");
}

__device__ __forceinline__ int ld_acquire(const int32_t* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// Byte offset of 16-byte piece `ch` of row `r` inside a K-major tile with the 128-byte swizzle.
__device__ __forceinline__ uint32_t sw128(int r, int ch) { return (uint32_t)(r * 128 + ((ch ^ (r & 7)) << 4)); }

// ---------------------------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------------------------
struct TcArgs {
  const __nv_bfloat16* x;       // [T, H]
  const __nv_bfloat16* w_gate;  // [E + ns, I, H]
  const __nv_bfloat16* w_up;    // [E + ns, I, H]
  const __nv_bfloat16* w_down;  // [E + ns, I/16, H, 16]
  const int32_t* perm;          // slot ids grouped by expert
  const float* topk_w;          // [T, k]
  const WorkItem* items;
  const int32_t* n_items;
  __nv_bfloat16* act_g;         // [items][NT][I] published activations
  int32_t* win_flags;           // [items * I/64] groups published per window (zeroed by the selection kernel)
  float* y;                     // [T, H], pre-zeroed rows of computed tokens
  int32_t* status;
  Dims d;
};

// The sequence of operations a CTA performs on its group range [lo, hi); every warp role walks the
// same sequence.  Group indices are global (item * NG + group in item); since NG is a multiple of
// 4, window W = group >> 2 never straddles two items.
//
// A super-chunk covers up to scw windows.  When the whole range is one super-chunk (the usual case
// at small row counts) the groups of the windows it shares with its neighbours go first in phase 1
// and the full windows last, and phase 2 starts with the shared windows: every CTA publishes what
// its neighbours need early, and the exchange latency hides behind streaming.  With several
// super-chunks the order is ascending and the tiles of the head window come last of all.
enum { OP_P1 = 0, OP_PUBLISH = 1, OP_P2 = 2 };
struct Op {
  int kind;
  int item;     // P1, P2: work item (all groups of a tile belong to one item)
  int g;        // P1: number of groups (1..4)
  int grp[4];   // P1: their global indices
  int tile;     // P1: accumulator index inside the super-chunk
  int W;        // P2: global window index
  int a, b;     // P2: the CTA's groups [a, b) of the window (0..4)
};

struct Walker {
  int lo, hi, NG, HT, scw;
  int s_lo, s_hi, nH, nT, nM, tail0, mid0, li, ji, tile, state;
  int item0, base0;     // item of the super-chunk's first group and that item's first group
  bool single, deferred;
  __device__ Walker(int lo_, int hi_, int ng, int ht, int sc_windows)
      : lo(lo_), hi(hi_), NG(ng), HT(ht), scw(sc_windows), s_lo(lo_), s_hi(lo_), nH(0), nT(0), nM(0), tail0(0),
        mid0(0), li(0), ji(0), tile(0), state(0), item0(lo_ / ng), base0((lo_ / ng) * ng), single(false),
        deferred(false) {}
  // item of a group at or after the super-chunk's first group (no division: a super-chunk spans few items)
  __device__ int item_of(int grp) const {
    int it = item0, b = base0 + NG;
    while (grp >= b) {
      b += NG;
      ++it;
    }
    return it;
  }
  // phase-1 order of the super-chunk: head part, tail part, middle
  __device__ int group_at(int i) const {
    return i < nH ? s_lo + i : (i < nH + nT ? tail0 + (i - nH) : mid0 + (i - nH - nT));
  }
  __device__ int lo_item() const {     // the deferred head job comes after the last super-chunk: count down
    int it = item0, b = base0;
    while (lo < b) {                   // never taken unless the walk moved past lo's item
      b -= NG;
      --it;
    }
    return it;
  }
  __device__ bool p2(Op& op, int w, int from, int to) const {
    op.kind = OP_P2;
    op.W = w;
    op.a = max(from, 4 * w) - 4 * w;
    op.b = min(to, 4 * w + 4) - 4 * w;
    op.item = w == (lo >> 2) ? lo_item() : item_of(4 * w);
    return op.a * HT / 4 < op.b * HT / 4;     // jobs without a tile are skipped
  }
  __device__ bool next(Op& op) {
    for (;;) {
      switch (state) {
        case 0:                                     // open the next super-chunk
          if (s_hi >= hi) { state = 4; break; }
          s_lo = s_hi;
          s_hi = min(hi, ((s_lo >> 2) + scw) << 2);
          while (s_lo >= base0 + NG) {              // item of the new first group
            base0 += NG;
            ++item0;
          }
          single = (s_lo == lo && s_hi == hi);
          if (single) {
            nH = (s_lo & 3) ? min(s_hi, (s_lo | 3) + 1) - s_lo : 0;
            tail0 = max(s_hi & ~3, s_lo + nH);
            nT = (s_hi & 3) ? max(0, s_hi - tail0) : 0;
            mid0 = s_lo + nH;
            nM = (s_hi - nT) - mid0;
          } else {
            nH = nT = 0;
            mid0 = s_lo;
            nM = s_hi - s_lo;
            tail0 = s_hi;
          }
          li = 0;
          ji = 0;
          tile = 0;
          state = 1;
          break;
        case 1: {                                   // phase-1 tiles: up to 4 groups of one item, shared groups apart
          const int n = nH + nT + nM;
          if (li >= n) { state = 2; break; }
          const int first = group_at(li);
          const int first_item = item_of(first);
          int g = 1;
          while (g < 4 && li + g < n && li + g != nH + nT && item_of(group_at(li + g)) == first_item) ++g;
          op.kind = OP_P1;
          op.item = first_item;
          op.g = g;
#pragma unroll
          for (int q = 0; q < 4; ++q) op.grp[q] = q < g ? group_at(li + q) : first;
          op.tile = tile++;
          li += g;
          return true;
        }
        case 2:
          op.kind = OP_PUBLISH;
          state = 3;
          return true;
        case 3: {                                   // phase-2 jobs, one per window touched
          if (single) {
            const int n_mid = (nM + 3) >> 2;
            const int n_jobs = (nT > 0) + (nH > 0) + n_mid;
            if (ji >= n_jobs) { state = 0; break; }
            int j = ji++;
            int w;
            if (nT > 0 && j == 0) w = (s_hi - 1) >> 2;
            else {
              j -= (nT > 0);
              if (nH > 0 && j == 0) w = s_lo >> 2;
              else w = (mid0 >> 2) + j - (nH > 0);
            }
            if (p2(op, w, s_lo, s_hi)) return true;
          } else {
            const int w = (s_lo >> 2) + ji;
            if (w > ((s_hi - 1) >> 2)) { state = 0; break; }
            ++ji;
            if (w == (lo >> 2) && (lo & 3) != 0) { deferred = true; break; }
            if (p2(op, w, s_lo, s_hi)) return true;
          }
          break;
        }
        case 4:                                     // the head window, shared with the previous CTA, comes last
          state = 5;
          if (deferred && p2(op, lo >> 2, lo, hi)) return true;
          break;
        default:
          return false;
      }
    }
  }
};

// The stages of the loader -> tensor-core ring, derived from the operation sequence.  The ring is
// byte-granular: a stage takes what its tile needs (a 1-group tile a quarter of a 4-group tile), so
// the bytes in flight do not shrink with the tile.  Placement is a pure function of the sequence;
// the loaders and the MMA warp compute it independently.
struct Stage {
  int kind;            // OP_P1, OP_P2 or OP_PUBLISH (no bytes)
  bool first, last;    // first / last stage of its operation
  int k0, n;           // P1: first k-block, k-blocks;  P2: first W_down tile, tiles
  uint32_t off;        // byte offset in the ring
  uint32_t len;        // bytes reserved (including what a partial tile's 128-row reads run past its end)
  uint32_t it, lap;    // running stage index; how often the ring wrapped before this stage
};

template <int NT>
struct StageIter {
  using C = TcCfg<NT>;
  Walker walk;
  Op op;
  int KB, HT, pos, end;
  bool have_op;
  uint32_t cur, it, lap;
  __device__ StageIter(int lo, int hi, int ng, int kb, int ht)
      : walk(lo, hi, ng, ht, C::kScWindows), KB(kb), HT(ht), pos(0), end(0), have_op(false), cur(0), it(0), lap(0) {}
  __device__ bool next(Stage& st) {
    if (!have_op) {
      if (!walk.next(op)) return false;
      if (op.kind == OP_PUBLISH) {
        st.kind = OP_PUBLISH;
        return true;
      }
      have_op = true;
      pos = op.kind == OP_P1 ? 0 : op.a * HT / 4;
      end = op.kind == OP_P1 ? KB : op.b * HT / 4;
      st.first = true;
    } else {
      st.first = false;
    }
    st.kind = op.kind;
    st.k0 = pos;
    st.n = min(C::kKbs, end - pos);
    pos += C::kKbs;
    st.last = pos >= end;
    uint32_t bytes, over;
    if (op.kind == OP_P1) {
      bytes = (uint32_t)C::kKbs * (4096u * op.g + C::kBSub);
      over = (uint32_t)(128 - 32 * op.g) * 128u;
    } else {
      bytes = (uint32_t)st.n * kATileBytes;
      over = 0;
    }
    // Large stages sit on a grid of full-stage slots, so that the ring always holds as many of them as
    // fit (small stages placed before them would otherwise leave the last slot a few KB short).
    if (2 * bytes > (uint32_t)C::kStageBytes) cur = (cur + C::kStageBytes - 1) / C::kStageBytes * C::kStageBytes;
    if (cur + bytes + over > (uint32_t)C::kRingBytes) {
      cur = 0;
      ++lap;
    }
    st.off = cur;
    st.len = bytes + over;
    st.lap = lap;
    st.it = it++;
    cur += bytes;
    if (st.last) have_op = false;
    return true;
  }
};

template <int NT>
__global__ void __launch_bounds__(kTcThreads, 1)
k_experts_tc(TcArgs a) {
  using C = TcCfg<NT>;
  constexpr bool RES = C::kRes;
  constexpr int KBS = C::kKbs;
  constexpr int NB = kRingBars;
  extern __shared__ unsigned char smem_dyn[];
  const Dims d = a.d;
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  unsigned char* act_buf = smem + C::kRingBytes;                                 // [kActBufs][NT][128 B]
  uint64_t* bars = reinterpret_cast<uint64_t*>(act_buf + C::kActBufs * C::kActBytes);
  uint64_t* bar_full = bars;                                       // [NB] loaders -> MMA
  uint64_t* bar_empty = bars + NB;                                 // [NB] MMA -> loaders
  uint64_t* bar_acc1_full = bars + 2 * NB;                         // [kScWindows]
  uint64_t* bar_acc1_empty = bar_acc1_full + C::kScWindows;        // [1]
  uint64_t* bar_act_full = bar_acc1_empty + 1;                     // [kActBufs]
  uint64_t* bar_act_empty = bar_act_full + C::kActBufs;            // [kActBufs]
  uint64_t* bar_acc2_full = bar_act_empty + C::kActBufs;           // [kAcc2]
  uint64_t* bar_acc2_empty = bar_acc2_full + C::kAcc2;             // [kAcc2]
  int32_t* tbl_row = reinterpret_cast<int32_t*>(reinterpret_cast<unsigned char*>(bars) + C::kBarBytes);   // [4][NT]
  float* tbl_wt = reinterpret_cast<float*>(tbl_row + 4 * NT);                                             // [4][NT]
  int32_t* ld_row = reinterpret_cast<int32_t*>(tbl_wt + 4 * NT);                                          // [kLoaders][NT]
  uint4* ld_queue = reinterpret_cast<uint4*>(ld_row + kLoaders * NT);                                     // [kLoaders][kRingBars]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ld_queue + kLoaders * kRingBars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int KB = d.H / 64;          // k-blocks of phase 1
  const int HT = d.H / 128;         // row tiles of W_down
  const int NG = d.I / kGroupCols;  // groups per work item
  const int WPI = NG / 4;           // windows per work item

  if (threadIdx.x == 0) {
    for (int s = 0; s < NB; ++s) {
      mbar_init(smem_u32(bar_full + s), kLoaders * 32);
      mbar_init(smem_u32(bar_empty + s), 1);
    }
    for (int i = 0; i < C::kScWindows; ++i) mbar_init(smem_u32(bar_acc1_full + i), 1);
    mbar_init(smem_u32(bar_acc1_empty), 4);
    for (int i = 0; i < C::kActBufs; ++i) {
      mbar_init(smem_u32(bar_act_full + i), 32);
      mbar_init(smem_u32(bar_act_empty + i), 1);
    }
    for (int i = 0; i < C::kAcc2; ++i) {
      mbar_init(smem_u32(bar_acc2_full + i), 1);
      mbar_init(smem_u32(bar_acc2_empty + i), 4);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kMmaWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"((uint32_t)C::kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // Everything above overlaps the selection kernel (programmatic dependent launch); its tables are
  // complete and visible from here on.
  asm volatile("griddepcontrol.wait;" ::: "memory");

  // This CTA's contiguous range of groups.
  const long long n_groups = (long long)(*a.n_items) * NG;
  const int g_lo = (int)(n_groups * blockIdx.x / gridDim.x), g_hi = (int)(n_groups * (blockIdx.x + 1) / gridDim.x);

  if (warp < kLoaders) {
    // ------------------------------ loaders: weights and token rows into the ring ------------------------------
    constexpr int LPR = KBS * 8;            // lanes per row in phase 1 (16-byte pieces of KBS k-blocks)
    constexpr int RPI = 32 / LPR;           // rows per warp instruction
    constexpr int RSTEP = kLoaders * RPI;   // rows between two instructions of one warp
    const int sub = lane / LPR, kbi = (lane >> 3) % KBS, ch = lane & 7;
    int32_t* my_rows = ld_row + warp * NT;
    uint4* my_queue = ld_queue + warp * NB;     // (offset, lap, index) of this warp's stages in flight, oldest first
    int tbl_item = -1, in_flight = 0;
    uint32_t q_tail = 0;                        // running index of the oldest stage in flight
    bool ok = true;
    StageIter<NT> head(g_lo, g_hi, NG, KB, HT);
    Stage st;
    // Per tile (phase 1) or job (phase 2) this lane's source pointers are formed once; a stage then only
    // adds its k offset (phase 1) or steps to the next tile (phase 2).
    const __nv_bfloat16* src1[4][2];        // phase 1: [group][gate, up], this lane's first row and 16-byte piece
    const __nv_bfloat16* src2 = nullptr;    // phase 2: this lane's first row of the next W_down tile
    const int rr0 = warp * RPI + sub;       // phase 1: first row inside a 16-row block; the others follow RSTEP apart
    const uint32_t dst1 = (uint32_t)rr0 * 128u + (uint32_t)((ch ^ (rr0 & 7)) << 4);   // (RSTEP is a multiple of 8: same swizzle)
    // phase 2: W_down is stored in slabs of 16 columns ([I/16][H][16]); a window's 128-byte tile row is
    // gathered from four slabs.  Per instruction a warp copies 4 rows x 32 bytes from each of them.
    const uint64_t pol = stream_policy();
    const int r_first = warp * 4 + ((lane & 7) >> 1);
    const int ch2 = (lane >> 3) * 2 + (lane & 1);                                     // 16-byte piece of the tile row
    const uint32_t dst2 = sw128(r_first, ch2);
    const size_t rstep1 = (size_t)RSTEP * d.H, rstep2 = (size_t)(4 * kLoaders) * 16, tstep2 = (size_t)128 * 16;
    int ncols = 0;
#pragma unroll
    for (int q = 0; q < 4; ++q) src1[q][0] = src1[q][1] = nullptr;
    while (ok && head.next(st)) {
      if (st.kind == OP_PUBLISH) continue;
      // make room: the oldest stages in flight are released by the MMA warp in order
      while (in_flight > 0) {
        const uint4 ts = my_queue[q_tail % NB];   // x: offset, y: lap
        const bool conflict = in_flight >= NB || ts.y + 1 < st.lap || (ts.y + 1 == st.lap && ts.x < st.off + st.len);
        if (!conflict) break;
        if (!(ok = mbar_wait_warp<64>(smem_u32(bar_empty + q_tail % NB), (q_tail / NB) & 1, abort_flag, a.status, 1))) break;
        ++q_tail;
        --in_flight;
      }
      if (!ok) break;
      if (lane == 0) my_queue[st.it % NB] = make_uint4(st.off, st.lap, 0u, 0u);
      __syncwarp();
      const Op& op = head.op;
      const uint32_t base = smem_u32(smem) + st.off;
      if (st.kind == OP_P1) {
        if (st.first) {
          const WorkItem item = a.items[op.item];
          ncols = RES ? d.T : item.n;
          if (!RES && op.item != tbl_item) {
            __syncwarp();
            for (int r = lane; r < item.n; r += 32) {
              int row;
              float wt;
              slot_row_weight(a.perm[item.begin + r], d.T, d.k, a.topk_w, row, wt);
              my_rows[r] = row;
            }
            __syncwarp();
            tbl_item = op.item;
          }
          // row r of the tile = 16-row block (2 * group + (0: gate, 1: up)) * 16 + rr
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const size_t off = ((size_t)item.e * d.I + (size_t)(op.grp[q] - op.item * NG) * kGroupCols + rr0) * d.H +
                               kbi * 64 + ch * 8;
            src1[q][0] = a.w_gate + off;
            src1[q][1] = a.w_up + off;
          }
        }
        if (st.k0 + kbi < KB) {
          const uint32_t sub_bytes = 4096u * op.g;                     // one k-block of the tile
          const uint32_t dstA = base + kbi * sub_bytes + dst1;
          const int koff = st.k0 * 64;
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            if (q < op.g) {
#pragma unroll
              for (int m = 0; m < 2; ++m) {
#pragma unroll
                for (int ii = 0; ii < 16 / RSTEP; ++ii)
                  cp_async16_stream(dstA + (uint32_t)(((q * 2 + m) * 16 + ii * RSTEP) * 128), src1[q][m] + koff + ii * rstep1, pol);
              }
            }
          }
          const uint32_t dstB = base + KBS * sub_bytes + kbi * C::kBSub;
          for (int r = rr0; r < ncols; r += RSTEP)
            cp_async16(dstB + sw128(r, ch), a.x + (size_t)(RES ? r : my_rows[r]) * d.H + (koff + kbi * 64 + ch * 8));
        }
      } else {
        if (st.first) {
          const WorkItem item = a.items[op.item];
          src2 = a.w_down + (((size_t)item.e * NG + (op.W - op.item * WPI) * 4 + (ch2 >> 1)) * d.H +
                             (size_t)st.k0 * 128 + r_first) * 16 + (ch2 & 1) * 8;
        }
        for (int i = 0; i < st.n; ++i, src2 += tstep2) {
          const uint32_t dstA = base + i * kATileBytes + dst2;
#pragma unroll
          for (int ii = 0; ii < 128 / (4 * kLoaders); ++ii)
            cp_async16_stream(dstA + (uint32_t)(ii * 4 * kLoaders) * 128u, src2 + ii * rstep2, pol);
        }
      }
      cp_async_arrive(smem_u32(bar_full + st.it % NB));     // the stage is handed over when this lane's copies land
      ++in_flight;
    }
    // everything still in flight lands before shared memory is released (also on abort)
    cp_async_wait_all();
  } else if (warp == kMmaWarp) {
    // ------------------------------ MMA issuer (whole warp converged, elected lane issues) ------------------------------
    uint32_t sc_i = 0, t2 = 0, jc = 0, idesc = 0, ab = 0;
    uint64_t act_desc = 0;
    bool ok = true;
    StageIter<NT> si(g_lo, g_hi, NG, KB, HT);
    Stage st;
    while (ok && si.next(st)) {
      if (st.kind == OP_PUBLISH) { ++sc_i; continue; }
      const Op& op = si.op;
      const uint32_t base = smem_u32(smem) + st.off;
      if (st.first) {
        const WorkItem item = a.items[op.item];
        idesc = make_idesc_bf16(RES ? kResidentRows : ((item.n + 15) & ~15));
      }
      if (st.kind == OP_P1) {
        if (st.first && op.tile == 0) {
          // the epilogue has read the previous super-chunk's accumulators
          if (!(ok = mbar_wait_warp(smem_u32(bar_acc1_empty), (sc_i & 1) ^ 1, abort_flag, a.status, 3))) break;
          tc_fence_after();
        }
        if (!(ok = mbar_wait_warp(smem_u32(bar_full + st.it % NB), (st.it / NB) & 1, abort_flag, a.status, 4))) break;
        // The barrier fires when the loaders' cp.async copies have landed in shared memory (completion-
        // triggered arrival), so the tiles are in place for the tensor core without a further proxy fence.
        tc_fence_after();
        const uint32_t acc1 = tmem_base + op.tile * NT;
        const uint32_t sub_bytes = 4096u * op.g;
        for (int i = 0; i < st.n; ++i) {
          const uint64_t da = make_kmajor_sw128_desc(base + i * sub_bytes);
          const uint64_t db = make_kmajor_sw128_desc(base + KBS * sub_bytes + i * C::kBSub);
#pragma unroll
          for (int k4 = 0; k4 < 4; ++k4) tc_mma(acc1, da + 2 * k4, db + 2 * k4, idesc, ((st.k0 + i) | k4) != 0);
        }
        tc_commit(smem_u32(bar_empty + st.it % NB));
        if (st.last) tc_commit(smem_u32(bar_acc1_full + op.tile));
      } else {
        if (st.first) {
          ab = jc % C::kActBufs;
          if (!(ok = mbar_wait_warp(smem_u32(bar_act_full + ab), (jc / C::kActBufs) & 1, abort_flag, a.status, 6))) break;
          tc_fence_after();
          act_desc = make_kmajor_sw128_desc(smem_u32(act_buf + ab * C::kActBytes));
        }
        if (!(ok = mbar_wait_warp(smem_u32(bar_full + st.it % NB), (st.it / NB) & 1, abort_flag, a.status, 8))) break;
        for (int i = 0; i < st.n; ++i, ++t2) {
          const uint32_t b = t2 % C::kAcc2, u = t2 / C::kAcc2;
          if (!(ok = mbar_wait_warp(smem_u32(bar_acc2_empty + b), (u & 1) ^ 1, abort_flag, a.status, 7))) break;
          tc_fence_after();
          const uint64_t da = make_kmajor_sw128_desc(base + i * kATileBytes);
          const uint32_t acc2 = tmem_base + (C::kScWindows + b) * NT;
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) tc_mma(acc2, da + 2 * kk, act_desc + 2 * kk, idesc, kk != 0);
          tc_commit(smem_u32(bar_acc2_full + b));
        }
        if (!ok) break;
        tc_commit(smem_u32(bar_empty + st.it % NB));
        if (st.last) {
          tc_commit(smem_u32(bar_act_empty + ab));
          ++jc;
        }
      }
    }
  } else if (warp == kActWarp) {
    // ------------------------------ activation-window loader (B operand of phase 2) ------------------------------
    uint32_t jc = 0;
    bool ok = true;
    Walker walk(g_lo, g_hi, NG, HT, C::kScWindows);
    Op op;
    while (ok && walk.next(op)) {
      if (op.kind != OP_P2) continue;
      const WorkItem item = a.items[op.item];
      const uint32_t ab = jc % C::kActBufs;
      ok = mbar_wait<64>(smem_u32(bar_act_empty + ab), ((jc / C::kActBufs) & 1) ^ 1, abort_flag, a.status, 14);
      // all four groups of the window published (by this CTA and / or its neighbours)?
      if (ok && lane == 0) {
        const int32_t* flag = a.win_flags + op.W;
        if (ld_acquire(flag) < 4) {
          const unsigned long long t0 = clock64();
          while (ld_acquire(flag) < 4) {
            __nanosleep(64);
            if (*abort_flag) { ok = false; break; }
            if (clock64() - t0 > kWaitCycles) {
              *abort_flag = 1;
              set_status(a.status, TEAM_ERR_TIMEOUT, 15);
              ok = false;
              break;
            }
          }
        }
      }
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      const int ncols = RES ? d.T : item.n;
      const int w = op.W - op.item * WPI;
      const uint32_t dstB = smem_u32(act_buf + ab * C::kActBytes);
      const __nv_bfloat16* base = a.act_g + (size_t)op.item * NT * d.I + w * kWindowCols;
      for (int ch16 = lane; ch16 < ncols * 8; ch16 += 32) {
        const int r = ch16 >> 3, ch = ch16 & 7;
        cp_async16(dstB + sw128(r, ch), base + (size_t)r * d.I + ch * 8);
      }
      cp_async_commit();
      cp_async_wait_all();
      fence_async_smem();
      mbar_arrive(smem_u32(bar_act_full + ab));
      ++jc;
    }
  } else if (warp >= kEpiWarp0) {
    // ------------------------------ epilogue ------------------------------
    const int q = warp - kEpiWarp0;               // TMEM lane quarter == warp_id % 4
    int32_t* my_row = tbl_row + q * NT;
    float* my_wt = tbl_wt + q * NT;
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    uint32_t t2 = 0, use1 = 0;                    // use1: bit t = parity of accumulator t's full barrier
    int tbl_item = -1;
    bool ok = true;
    Walker walk(g_lo, g_hi, NG, HT, C::kScWindows);
    Op op;
    while (ok && walk.next(op)) {
      if (op.kind == OP_P1) {
        // ---- SwiGLU: TMEM -> registers -> bf16 activations in the global scratch ----
        const WorkItem item = a.items[op.item];
        const int ncols = RES ? d.T : item.n;
        ok = mbar_wait_warp<32>(smem_u32(bar_acc1_full + op.tile), (use1 >> op.tile) & 1, abort_flag, a.status, 10);
        if (!ok) break;
        use1 ^= 1u << op.tile;
        tc_fence_after();
        if (q < op.g) {
          int grp = op.grp[0];                     // this warp's group
#pragma unroll
          for (int i = 1; i < 4; ++i)
            if (i == q) grp = op.grp[i];
          const int col = (grp - op.item * NG) * kGroupCols + (lane & 15);   // intermediate column of this lane pair
          const bool is_gate = lane < 16;                                   // lanes 0-15 hold gate rows, 16-31 up rows
          __nv_bfloat16* dst = a.act_g + (size_t)op.item * NT * d.I + col;
          const uint32_t acc1 = tmem_base + op.tile * NT + lane_off;
          for (int c0 = 0; c0 < ncols; c0 += 8) {
            float v[8];
            tmem_ld8(acc1 + c0, v);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const float o = __shfl_xor_sync(0xffffffffu, v[j], 16);
              const float g = is_gate ? v[j] : o;
              const float u = is_gate ? o : v[j];
              v[j] = g / (1.f + expf(-g)) * u;
            }
            // lanes 0-15 store tokens c0..c0+3, lanes 16-31 store c0+4..c0+7
            const int jb = is_gate ? 0 : 4;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const int n = c0 + jb + j;
              if (n < ncols) dst[(size_t)n * d.I] = __float2bfloat16_rn(v[jb + j]);
            }
          }
          // this warp's group of the window is published: visible to every CTA before the count moves
          __syncwarp();
          if (lane == 0) {
            __threadfence();
            atomicAdd(a.win_flags + (grp >> 2), 1);
          }
        }
      } else if (op.kind == OP_PUBLISH) {
        // the super-chunk's accumulators are free again
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(bar_acc1_empty));
      } else {
        // ---- down projection tiles: scale by routing weight, add into y ----
        const WorkItem item = a.items[op.item];
        const int ncols = RES ? d.T : item.n;
        if (op.item != tbl_item) {
          __syncwarp();
          if (RES) {
            for (int c = lane; c < kResidentRows; c += 32) {
              my_row[c] = c;
              my_wt[c] = 0.f;
            }
            __syncwarp();
          }
          for (int r = lane; r < item.n; r += 32) {
            int row;
            float wt;
            slot_row_weight(a.perm[item.begin + r], d.T, d.k, a.topk_w, row, wt);
            if (RES) {
              my_wt[row] = wt;
            } else {
              my_row[r] = row;
              my_wt[r] = wt;
            }
          }
          __syncwarp();
          tbl_item = op.item;
        }
        const int ht1 = op.b * HT / 4;
        int ht = op.a * HT / 4;
        // Few columns: a tile's epilogue is one short tensor-memory load, so up to four tiles are taken per
        // round (their loads in flight together, one wait) instead of paying the load latency per tile.
        while (ncols <= 8 && ht < ht1) {
          const int nb = min(C::kAcc2 < 4 ? C::kAcc2 : 4, ht1 - ht);     // never more than the MMA warp can run ahead
          uint32_t r[4][8];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            if (i < nb && ok) {
              const uint32_t b = (t2 + i) % C::kAcc2, u = (t2 + i) / C::kAcc2;
              ok = mbar_wait_warp<32>(smem_u32(bar_acc2_full + b), u & 1, abort_flag, a.status, 11);
              if (ok) {
                tc_fence_after();
                tmem_ld8_issue(tmem_base + (C::kScWindows + b) * NT + lane_off, r[i]);
              }
            }
          }
          if (!ok) break;
          tmem_ld_wait(r[0], r[1], r[2], r[3]);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            if (i < nb) {
              float* ycol = a.y + (ht + i) * 128 + q * 32 + lane;
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                if (j < ncols) {
                  const float wt = my_wt[j];
                  if (wt != 0.f) atomicAdd(ycol + (size_t)my_row[j] * d.H, wt * __uint_as_float(r[i][j]));
                }
              }
            }
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0)
            for (int i = 0; i < nb; ++i) mbar_arrive(smem_u32(bar_acc2_empty + (t2 + i) % C::kAcc2));
          ht += nb;
          t2 += nb;
        }
        if (!ok) break;
        for (; ht < ht1; ++ht, ++t2) {
          const uint32_t b = t2 % C::kAcc2, u = t2 / C::kAcc2;
          ok = mbar_wait_warp<32>(smem_u32(bar_acc2_full + b), u & 1, abort_flag, a.status, 11);
          if (!ok) break;
          tc_fence_after();
          const uint32_t acc2 = tmem_base + (C::kScWindows + b) * NT + lane_off;
          float* ycol = a.y + ht * 128 + q * 32 + lane;
          for (int c0 = 0; c0 < ncols; c0 += 8) {
            float v[8];
            tmem_ld8(acc2 + c0, v);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const int n = c0 + j;
              if (n < ncols) {
                const float wt = my_wt[n];
                if (wt != 0.f) atomicAdd(ycol + (size_t)my_row[n] * d.H, wt * v[j]);
              }
            }
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(bar_acc2_empty + b));
        }
      }
    }
  }

  // ------------------------------ teardown ------------------------------
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)C::kTmemCols)
                 : "memory");
  }
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
// Rows per work item for a context: 16 selects the resident-N mode.
int experts_tc_item_tile(int max_rows) {
  if (max_rows <= kResidentRows) return 16;
  if (max_rows <= 64) return 32;
  if (max_rows <= 256) return 64;
  return 128;
}

template <int NT>
static cudaError_t launch_tc(TcArgs args, int grid, cudaStream_t s) {
  // Cooperative: CTAs that share a window wait for each other's activations, so all must be resident.
  // Programmatic serialization: the CTAs may start their prologue while the selection kernel still runs.
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kTcThreads);
  cfg.dynamicSmemBytes = (size_t)TcCfg<NT>::kSmemBytes;
  cfg.stream = s;
  cudaLaunchAttribute attrs[2];
  attrs[0].id = cudaLaunchAttributeCooperative;
  attrs[0].val.cooperative = 1;
  attrs[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attrs[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attrs;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, k_experts_tc<NT>, args);
}

template <int NT>
static cudaError_t configure_tc() {
  cudaError_t e = cudaFuncSetAttribute(k_experts_tc<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, TcCfg<NT>::kSmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(k_experts_tc<NT>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
  return e;
}

cudaError_t configure_experts_tc(int item_tile) {
  switch (item_tile) {
    case 16: return configure_tc<16>();
    case 32: return configure_tc<32>();
    case 64: return configure_tc<64>();
    case 128: return configure_tc<128>();
    default: return cudaErrorInvalidValue;
  }
}

cudaError_t launch_experts_tc(int item_tile, const void* x, const void* w_gate, const void* w_up, const void* w_down,
                              Workspace ws, float* y, Dims d, int grid, cudaStream_t s) {
  TcArgs a;
  a.x = static_cast<const __nv_bfloat16*>(x);
  a.w_gate = static_cast<const __nv_bfloat16*>(w_gate);
  a.w_up = static_cast<const __nv_bfloat16*>(w_up);
  a.w_down = static_cast<const __nv_bfloat16*>(w_down);
  a.perm = ws.r.perm;
  a.topk_w = ws.r.topk_w;
  a.items = ws.items;
  a.n_items = ws.n_items;
  a.act_g = ws.act_g;
  a.win_flags = ws.win_flags;
  a.y = y;
  a.status = ws.status;
  a.d = d;
  switch (item_tile) {
    case 16: return launch_tc<16>(a, grid, s);
    case 32: return launch_tc<32>(a, grid, s);
    case 64: return launch_tc<64>(a, grid, s);
    case 128: return launch_tc<128>(a, grid, s);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace team
