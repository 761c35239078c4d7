// Weight-streaming expert kernel (bf16 weights, hidden size 1024 or 2048).
//
// With a handful of rows per expert the SwiGLU experts (Eq. 1) are a matrix-vector problem: ~1 MB of weights
// per SM and a few hundred kFLOP.  Staging tiles for the tensor-memory path costs more in hand-offs between
// warps than the math is worth, so here every warp is its own pipeline: it copies 2 KB chunks of weights from
// HBM into a private ring in shared memory with asynchronous copies, several chunks ahead, and multiplies each
// chunk with the token rows using warp-level mma (m16n8k16: 16 weight rows x 8 tokens).  No warp waits for
// another one inside a phase, and no CTA ever waits for another CTA.
//
// Work partition: the intermediate dimension of every activated expert (or work item of an expert) is cut
// into groups of 16 columns, the global list of groups into one contiguous range per CTA.  A group is
// self-contained: its 16 gate rows and 16 up rows of W give 16 activations per token (phase 1), and those
// multiply the group's slab of W_down, 16 columns of all H rows, stored contiguously ([I/16][H][16]), into a
// partial y that is added to the output with fp32 reductions (phase 2).  Groups are handled in passes of up
// to 8 (4 with 16 token columns):
//
//   phase 1   warp = (gate | up tile of 16 rows) x (one of 8 slices of the hidden dimension), for every
//             group of the pass in turn; chunk = 16 rows x 128 bytes; partial sums of a slice go to
//             shared memory.
//   barrier   sum the 8 slices, a = silu(gate) * up, round to bf16, keep in shared memory.
//   phase 2   warp = H/16 consecutive output rows, 64 at a time, for every group of the pass in turn;
//             chunk = 64 slab rows x 32 bytes; the accumulators stay in registers across the groups of one
//             expert and are scaled by the routing weights and added to y when the expert changes.
//
// A warp's copies run ahead across the barrier: while the slices are being summed, its first slab chunks of
// phase 2 are already on their way.
//
// Token columns.  Up to 8 rows per call: the call's rows themselves, for every expert (weight 0 where a row
// did not choose it), and the activated set is formed here from the rows' choices.  More rows: work items
// of 8 or 16 token-slots of one expert, built by the selection kernel, gathered into shared memory per item.
//
// Fused step (up to 8 rows, no dispatch table asked for).  The whole layer step is this one kernel: every CTA
// first computes the router logits of "its" experts (expert e on CTA e mod grid: the 4*E*H bytes of router
// weights are read once, spread over the SMs), the CTAs meet at a grid-wide barrier (cooperative launch, one
// arrival counter, bounded spin), and then every CTA repeats the tiny selection for the call's rows by itself
// from the T*E logits (Eq. 4, the two routing rounds of Algorithm 1, one warp per row) instead of waiting for
// a selection kernel: no second and third launch, no dependency hop between them.  CTA 0 writes the exports.
#include "team_common.cuh"
#include "team_topk.cuh"

namespace team {

constexpr int kStThreads = 512;
constexpr int kStWarps = 16;
constexpr int kStSlices = 8;                    // slices of the hidden dimension in phase 1
constexpr int kStRows = 8;                      // token rows (n of the mma)
constexpr int kStPassGroups = 8;                // groups whose partial sums fit in shared memory
constexpr int kStSlots = 4;                     // chunks per warp ring
constexpr int kStChunkBytes = 2048;
constexpr int kStRedBytes = kStPassGroups * kStSlices * 2 * 16 * kStRows * 4;

struct StArgs {
  const __nv_bfloat16* x;       // [T, H]
  const __nv_bfloat16* w_gate;  // [E + ns, I, H]
  const __nv_bfloat16* w_up;
  const __nv_bfloat16* w_down;  // [E + ns, I/16, H, 16]
  const int32_t* perm;
  const int32_t* topk_idx;      // [T, k] expert chosen per slot (-1: row skipped)
  const uint8_t* tok_class;     // [T]
  const float* topk_w;
  const WorkItem* items;
  const int32_t* n_items;
  float* y;                     // [T, H]
  Dims d;
  // fused step only: router and selection run inside the kernel
  const float* w_router;        // [E, H] fp32
  float* logits;                // [T, E] scratch (context workspace)
  StepPtrs st;
  Policy p;
  RoutePtrs r;                  // context tables (choices, classes, E_A) written by CTA 0
  RoutePtrs ex;                 // caller's exports, members may be null
  unsigned long long* arrivals; // grid barrier: counts CTA arrivals over all launches, never reset
  int32_t* status;
  long long spin_cycles;        // limit of the barrier's wait
  int extra_arrivals;           // diagnostic: arrivals the barrier waits for beyond the grid's own (0 in normal use)
  float* ordered;               // ordered combine: [grid][T][H] per-CTA partial outputs (null: fp32 reductions into y)
};

__device__ __forceinline__ uint32_t st_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
// Weights are read once per step: they are marked evict-first in L2 so that streaming them does not push out
// what the step's small kernels reuse from one step to the next (router weights, tables, code).
__device__ __forceinline__ uint64_t st_stream_policy() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void st_cp16(uint32_t dst, const void* src, uint64_t pol) {
  asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "l"(pol) : "memory");
}
__device__ __forceinline__ void st_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void st_wait_group() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void st_ldmatrix4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr)
               : "memory");
}
__device__ __forceinline__ uint4 st_ldg_stream(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}
// d += A(16x16, rows g / g+8) * B(16x8), bf16 inputs, fp32 accumulate
__device__ __forceinline__ void st_mma(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Position of the n-th (0-based) set bit of m; popcount(m) > n.  Five halvings instead of a bit-by-bit walk.
__device__ __forceinline__ int st_nth_set_bit(uint32_t m, int n) {
  int pos = 0;
#pragma unroll
  for (int width = 16; width >= 1; width >>= 1) {
    const int c = __popc(m & (((1u << width) - 1u) << pos));
    if (n >= c) {
      n -= c;
      pos += width;
    }
  }
  return pos;
}

// shared memory: token rows | partial sums [group][slice][gate, up][16 rows][tokens] | per-warp rings.
// ntl = token tiles of 8 (1 or 2): with 16 tokens a pass holds half the groups and a ring one slot less.
__host__ __device__ inline int stream_slots(int ntl) { return ntl == 1 ? kStSlots : kStSlots - 1; }
// The fused step keeps the rows' choices and a little scratch in shared memory; a pass of 7 groups instead
// of 8 makes the room.
constexpr int kStFusedPass = kStPassGroups - 1;
constexpr int kStFusedScratch = kStRedBytes / kStPassGroups;      // what the eighth group's partial sums took
__host__ __device__ inline size_t stream_red_bytes(bool fused) {
  return fused ? (size_t)kStRedBytes / kStPassGroups * kStFusedPass : (size_t)kStRedBytes;
}
__host__ __device__ inline size_t stream_smem_bytes(int H, int ntl, bool fused = false) {
  return (size_t)kStRows * ntl * H * 2 + stream_red_bytes(fused) + (size_t)kStWarps * stream_slots(ntl) * kStChunkBytes +
         (fused ? kStFusedScratch : 0);
}

__device__ __forceinline__ unsigned long long st_ld_acquire(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}

// CPG: 64-row chunks of a W_down slab per warp and group (H = CPG * 1024).
// GATHER = false: the call has at most 8 rows; all of them are the mma's token columns for every expert, and a
//                 row that did not choose the expert gets weight 0.
// GATHER = true:  any number of rows; work items of at most 8 * NTL token-slots of one expert (built by the
//                 selection kernel); a pass stays inside one item and the item's rows are gathered into shared
//                 memory.  NTL = 2 (two token tiles per weight fragment) halves how often an expert that many
//                 rows chose is streamed; its pass holds 4 groups instead of 8.
// FUSED = true (resident mode only): router logits, grid barrier and selection run in this kernel's prologue.
template <int CPG, bool GATHER, int NTL, bool FUSED = false>
__global__ void __launch_bounds__(kStThreads, 1) k_experts_stream(StArgs a) {
  static_assert(NTL == 1 || (NTL == 2 && GATHER), "two token tiles only in gather mode");
  static_assert(!FUSED || !GATHER, "the fused step keeps all rows resident");
  constexpr int TOK = kStRows * NTL;                 // token columns
  constexpr int PASS = FUSED ? kStFusedPass : kStPassGroups / NTL;          // groups per pass
  extern __shared__ __align__(128) unsigned char st_smem[];
  __shared__ __align__(16) __nv_bfloat16 s_act[PASS * TOK * 16];               // a = silu(gate) * up of the pass: [group][token][16]
  __shared__ float s_w[kStPassGroups][kStRows];                                // routing weight of token n for group q's expert
  __shared__ int s_item[kStPassGroups];
  __shared__ int s_row[TOK];            // gather: output row of token column n (-1: unused column)
  __shared__ float s_wt[TOK];           // gather: its routing weight
  constexpr int SLOTS = NTL == 1 ? kStSlots : kStSlots - 1;
  constexpr int H = CPG * 1024, HW = H / kStWarps;      // output rows per warp in phase 2
  constexpr int KS = H / kStSlices, NCH = KS / 64;      // phase 1: elements per slice, 64-wide chunks per slice
  const Dims d = a.d;
  const int I = d.I, T = d.T;
  unsigned char* xs = st_smem;                                                    // [TOK][H] bf16, 16-byte pieces swizzled
  float* red = reinterpret_cast<float*>(st_smem + (size_t)TOK * H * 2);          // [group][slice][2][16][TOK]
  constexpr size_t RED_BYTES = FUSED ? (size_t)kStRedBytes / kStPassGroups * kStFusedPass : (size_t)kStRedBytes;
  // fused step: the rows' choices, weights and classes live here for the whole launch
  unsigned char* fz = st_smem + (size_t)TOK * H * 2 + RED_BYTES + (size_t)kStWarps * SLOTS * kStChunkBytes;
  int32_t* f_idx = reinterpret_cast<int32_t*>(fz);                 // [T * k] (<= 128)
  float* f_wt = reinterpret_cast<float*>(fz + 512);                // [T * k]
  float* f_part = reinterpret_cast<float*>(fz + 1024);             // [warps][8] router partial sums
  uint32_t* f_mask = reinterpret_cast<uint32_t*>(fz + 1536);       // [8 group slots][8 words] E_A
  uint8_t* f_cls = fz + 1792;                                      // [8]
  int32_t* f_gslot = reinterpret_cast<int32_t*>(fz + 1808);        // [8] first row of the row's group
  int32_t* f_flag = reinterpret_cast<int32_t*>(fz + 1840);         // [1] barrier gave up
  const int32_t* c_idx = FUSED ? f_idx : a.topk_idx;
  const float* c_wt = FUSED ? f_wt : a.topk_w;
  const uint8_t* c_cls = FUSED ? f_cls : a.tok_class;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, c = lane & 3;        // fragment row (and token of the B fragment), k / token pair
  const int NG = I / 16;

  // ---- token rows into shared memory (an input of the call: may overlap the selection kernel) ----
  constexpr int per_row = H / 8;
  constexpr int kXLoads = TOK * per_row / kStThreads;         // 16-byte pieces per thread
  uint4 xv[kXLoads];
  // fused step: this CTA's first router weight row is requested ahead of everything (weights are never an
  // output of the preceding kernel); warp w owns H/16 consecutive elements, RV of them per lane
  constexpr int RV = H / (kStWarps * 32);                     // 4 (H = 2048) or 2 (H = 1024)
  float rw[4] = {0.f, 0.f, 0.f, 0.f};
  const int h_lane = warp * (H / kStWarps) + lane * RV;       // first hidden element of this lane
  auto load_router_row = [&](int e) {
    const float* src = a.w_router + (size_t)e * H + h_lane;
    if constexpr (RV == 4) {
      const float4 v = __ldg(reinterpret_cast<const float4*>(src));
      rw[0] = v.x; rw[1] = v.y; rw[2] = v.z; rw[3] = v.w;
    } else {
      const float2 v = __ldg(reinterpret_cast<const float2*>(src));
      rw[0] = v.x; rw[1] = v.y;
    }
  };
  if constexpr (FUSED) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next kernel may be scheduled behind this one
    if ((int)blockIdx.x < d.E) load_router_row(blockIdx.x);
    asm volatile("griddepcontrol.wait;" ::: "memory");               // x and y may come from / go to the preceding kernel
  }
  if (!GATHER) {
#pragma unroll
    for (int i = 0; i < kXLoads; ++i) {
      const int idx = tid + i * kStThreads, n = idx / per_row, ci = idx - n * per_row;
      xv[i] = n < T ? st_ldg_stream(a.x + (size_t)n * H + ci * 8) : make_uint4(0u, 0u, 0u, 0u);
    }
  }
  int e_slot[4] = {-1, -1, -1, -1};      // expert of slots lane, lane + 32, ... (T * k <= 128)
  if constexpr (!FUSED) {
    asm volatile("griddepcontrol.wait;" ::: "memory");     // the selection kernel's tables are complete from here on
    // the rows' choices (resident mode) are requested before the token rows are parked in shared memory, so that
    // the two round trips overlap when this kernel did not get to start ahead of the selection kernel's end
    if (!GATHER) {
#pragma unroll
      for (int b = 0; b < 4; ++b)
        if (b * 32 + lane < T * d.k) e_slot[b] = a.topk_idx[b * 32 + lane];
    }
  }
  // fused step: the step state of row `lane` (every warp holds a copy)
  int f_state = TEAM_TOK_CACHED, f_pos = 0, f_group = 0, f_branch = 0;
  float f_conf = 0.f;
  if constexpr (FUSED) {
    if (lane < T) {
      f_state = a.st.tok_state[lane];
      f_conf = a.st.conf[lane];
      f_pos = a.st.pos[lane];
      f_group = a.st.group[lane];
      f_branch = a.st.branch[lane];
    }
  }
  if (!GATHER) {
#pragma unroll
    for (int i = 0; i < kXLoads; ++i) {
      const int idx = tid + i * kStThreads, n = idx / per_row, ci = idx - n * per_row;
      *reinterpret_cast<uint4*>(xs + (size_t)n * H * 2 + ((ci ^ n) << 4)) = xv[i];
    }
  }
  // fused step, thread 0: the barrier's target, from the arrival count as it stands before this CTA arrives.  The
  // count is a multiple of the grid size between launches (every launch adds exactly one arrival per CTA), so
  // whatever this launch's other CTAs have added already, rounding down gives the launch's base.
  unsigned long long bar_target = 0ull;
  if constexpr (FUSED) {
    if (tid == 0) {
      const unsigned long long n = gridDim.x;
      bar_target = (st_ld_acquire(a.arrivals) / n + 1ull) * n + (unsigned long long)a.extra_arrivals;
    }
    // the output rows that will be accumulated into start from zero: the CTAs share the job
    {
      const uint32_t skip_rows = (a.p.flags & TEAM_F_DCD) ? __ballot_sync(0xffffffffu, lane < T && f_state == TEAM_TOK_CACHED) : 0u;
      const int total4 = T * H / 4;
      for (int i = blockIdx.x * kStThreads + tid; i < total4; i += gridDim.x * kStThreads) {
        const int t = (i * 4) / H;
        if (!((skip_rows >> t) & 1u)) reinterpret_cast<float4*>(a.y)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
    if (a.ordered != nullptr) {
      float4* mine = reinterpret_cast<float4*>(a.ordered + (size_t)blockIdx.x * T * H);
      for (int i = tid; i < T * H / 4; i += kStThreads) mine[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    if (tid < 64) f_mask[tid] = 0u;
    if (tid == 64) *f_flag = 0;
  }
  __syncthreads();

  // ---- this warp's ring and its fixed lane roles (nothing here depends on the selection: set up ahead of it) ----
  const uint32_t ring = st_smem_u32(st_smem + (size_t)TOK * H * 2 + RED_BYTES + (size_t)warp * SLOTS * kStChunkBytes);
  // phase-1 chunk: 16 rows x 128 bytes; lane copies one 16-byte piece of rows cp_row + 4j; piece p of row r sits at p ^ (r & 7)
  const int cp_row = lane >> 3, cp_piece = lane & 7;
  const uint32_t cp_off0 = cp_row * 128 + ((cp_piece ^ cp_row) << 4);          // rows cp_row, cp_row + 8 (+1024)
  const uint32_t cp_off1 = (cp_row + 4) * 128 + ((cp_piece ^ (cp_row + 4)) << 4);
  // phase-2 chunk: 64 slab rows x 32 bytes, contiguous in memory; lane copies pieces lane + 32j; half p of row r sits at p ^ bit 2 of r
  const uint32_t cq_off = (lane >> 1) * 32 + (((lane & 1) ^ ((lane >> 3) & 1)) << 4);
  // ldmatrix lane roles: A tile row and k half (low / high 8), B token row and k piece
  const int a_row = (lane & 7) + ((lane >> 3) & 1) * 8, a_hi = lane >> 4;
  const uint32_t a1_base = a_row * 128;
  const int a1_swz = a_row & 7;
  const uint32_t a2_off = a_row * 32 + ((a_hi ^ ((a_row >> 2) & 1)) << 4);
  const int b_tok = lane & 7, b_m = lane >> 3;
  const uint32_t xs_lane = st_smem_u32(xs) + (uint32_t)b_tok * H * 2;
  const int tile = warp & 1, ks = warp >> 1;     // phase 1: this warp's 16-row tile (gate | up) and hidden slice
  const __nv_bfloat16* wmat = tile ? a.w_up : a.w_gate;
  const uint64_t pol = st_stream_policy();

  // fused step: logits of the row this warp routes (warps 0 .. T-1), as order-preserving keys and as values
  uint32_t f_key[kMaxPerLane];
  int f_slot[kMaxPerLane];
  float f_val[kMaxPerLane];
  float f_margin = __builtin_huge_valf();
  int f_mycls = TEAM_CLS_SKIP;
  if constexpr (FUSED) {
    // ---- router logits of this CTA's experts: fp32 dot products over the staged rows ----
    const int E = d.E;
    for (int e = blockIdx.x; e < E; e += gridDim.x) {
      if (e != (int)blockIdx.x) load_router_row(e);
      float acc[kStRows];
#pragma unroll
      for (int n = 0; n < kStRows; ++n) {
        acc[n] = 0.f;
        if (n < T) {
          // RV bf16 elements of row n starting at h_lane: inside one 16-byte piece (RV divides 8)
          const unsigned char* px = xs + (size_t)n * H * 2 + ((((h_lane >> 3) ^ n)) << 4) + (h_lane & 7) * 2;
          if constexpr (RV == 4) {
            const uint2 v = *reinterpret_cast<const uint2*>(px);
            const float2 lo = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v.x));
            const float2 hi = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v.y));
            acc[n] = fmaf(rw[0], lo.x, acc[n]);
            acc[n] = fmaf(rw[1], lo.y, acc[n]);
            acc[n] = fmaf(rw[2], hi.x, acc[n]);
            acc[n] = fmaf(rw[3], hi.y, acc[n]);
          } else {
            const uint32_t v = *reinterpret_cast<const uint32_t*>(px);
            const float2 lo = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v));
            acc[n] = fmaf(rw[0], lo.x, acc[n]);
            acc[n] = fmaf(rw[1], lo.y, acc[n]);
          }
          acc[n] = warp_sum(acc[n]);
        }
      }
      if (lane == 0) {
#pragma unroll
        for (int n = 0; n < kStRows; ++n) f_part[warp * kStRows + n] = acc[n];
      }
      __syncthreads();
      if (tid < T) {
        float sum = 0.f;
#pragma unroll
        for (int w = 0; w < kStWarps; ++w) sum += f_part[w * kStRows + tid];      // fixed order
        a.logits[(size_t)tid * E + e] = sum;
      }
      __syncthreads();
    }
    // ---- grid barrier: every CTA's logits (and zeroed output rows) are visible behind it.  Thread 0 arrives
    //      and polls; meanwhile warp 1 classifies the rows (Eq. 4 needs no logits) and CTA 0 clears E_A's table ----
    if (tid == 0) {
      __threadfence();
      atomicAdd(a.arrivals, 1ull);
      const long long t_begin = clock64();
      while (st_ld_acquire(a.arrivals) < bar_target) {
        if (clock64() - t_begin > a.spin_cycles) {
          *f_flag = 1;
          break;
        }
      }
    }
    if (warp == 1) {
      if (lane < T && (f_group < 0 || f_group >= d.G || f_branch < 0 || f_branch > 255)) {
        if (blockIdx.x == 0) set_status(a.status, TEAM_ERR_STATE, 1);
        f_group = min(max(f_group, 0), d.G - 1);
        f_branch = min(max(f_branch, 0), 255);
      }
      const bool decoded = f_state == TEAM_TOK_NEW || f_state == TEAM_TOK_CACHED;
      const int lim = a.p.inclusive ? a.p.L_hot : a.p.L_hot - 1;      // |pos - j| <= lim
      bool near = a.p.prefix_decoded && f_pos + 1 <= lim;
      int gslot = lane;
      for (int v = T - 1; v >= 0; --v) {
        const int gv = __shfl_sync(0xffffffffu, f_group, v), bv = __shfl_sync(0xffffffffu, f_branch, v);
        const int pv = __shfl_sync(0xffffffffu, f_pos, v);
        const bool dv = __shfl_sync(0xffffffffu, (int)decoded, v) != 0;
        if (gv == f_group) {
          gslot = v;                                                     // ends at the group's first row
          if (bv == f_branch && dv && abs(f_pos - pv) <= lim) near = true;
        }
      }
      int cls;
      if (f_state == TEAM_TOK_CACHED) cls = (a.p.flags & TEAM_F_DCD) ? TEAM_CLS_SKIP : TEAM_CLS_FIRST;
      else if (f_state == TEAM_TOK_NEW || !(a.p.flags & TEAM_F_LAC)) cls = TEAM_CLS_FIRST;
      else cls = (f_conf > a.p.tau_hot || near) ? TEAM_CLS_FIRST : TEAM_CLS_COLD;
      if (lane >= T) cls = TEAM_CLS_SKIP;
      // a group with no first-round row: its masked rows are all routed freely
      bool has_first = false;
      for (int v = 0; v < T; ++v) {
        const int gv = __shfl_sync(0xffffffffu, f_group, v), cv = __shfl_sync(0xffffffffu, cls, v);
        if (gv == f_group && cv == TEAM_CLS_FIRST) has_first = true;
      }
      if (cls == TEAM_CLS_COLD && !has_first) cls = TEAM_CLS_FIRST;
      if (lane < kStRows) {
        f_cls[lane] = (uint8_t)cls;
        f_gslot[lane] = gslot;
      }
    }
    if (blockIdx.x == 0 && tid >= 64) {
      // E_A of groups nobody belongs to is empty: the table is cleared before the present groups are filled in
      const int n_words64 = (E + 63) / 64;
      for (int i = tid - 64; i < d.G * n_words64; i += kStThreads - 64) {
        a.r.group_mask[i] = 0ull;
        if (a.ex.group_mask) a.ex.group_mask[i] = 0ull;
      }
    }
    __syncthreads();
    if (*f_flag) {
      // the wait ran out: nothing of the step is computed, the status word says so
      if (tid == 0) set_status(a.status, TEAM_ERR_TIMEOUT, 20);
      return;
    }
    // ---- Algorithm 1, first round: one warp per row.  Only the picks are on the way to the first weight
    //      bytes: the activated set is the union of the first-round choices (cold rows add nothing to it), so
    //      the second round, the softmax and the routing weights wait until the first copies are in flight ----
    const int k = d.k, ne = (E + 31) / 32;
    if (warp < T) {
      const int t = warp;
      f_mycls = f_cls[t];
      if (f_mycls == TEAM_CLS_SKIP) {
        if (lane < k) {
          f_idx[t * k + lane] = -1;
          f_wt[t * k + lane] = 0.f;
        }
      } else {
#pragma unroll
        for (int i = 0; i < kMaxPerLane; ++i) {
          const int e = i * 32 + lane;
          f_val[i] = (i < ne && e < E) ? __ldcg(a.logits + (size_t)t * E + e) : kNegInf;      // written by other SMs: read from L2
          f_key[i] = float_key(f_val[i]);
          f_slot[i] = i;
        }
        if (f_mycls == TEAM_CLS_FIRST) {
          const int gs = f_gslot[t];
          sort_lane_keys(f_key, f_slot);
          const int n = warp_topk_picks(f_key, f_slot, k, lane,
                                        [&](int j, int e, uint32_t key) {
                                          f_idx[t * k + j] = e;
                                          f_wt[t * k + j] = key_float(key);       // the logit; turned into the weight later
                                          atomicOr(&f_mask[gs * 8 + (e >> 5)], 1u << (e & 31));
                                        },
                                        f_margin);
          if (n < k) {
            if (lane >= n && lane < k) f_idx[t * k + lane] = -1;
            if (blockIdx.x == 0 && lane == 0) set_status(a.status, TEAM_ERR_STATE, 3);
          }
        }
      }
    }
    __syncthreads();
  }

  // Resident mode needs no dispatch tables: with at most 8 rows every warp reads the rows' choices (T*k slots)
  // and forms the set of activated experts itself, word w of the bit set in lane w; activated expert number i
  // is the i-th set bit.
  int n_act = 0;
  uint32_t act_word = 0u;
  const int n_words = (d.E + d.ns + 31) >> 5;
  if (!GATHER) {
    if constexpr (FUSED) {
      // the union of the groups' necessary sets, straight from shared memory: word w in lane w
      if (lane < 8) {
#pragma unroll
        for (int gs = 0; gs < kStRows; ++gs) act_word |= f_mask[gs * 8 + lane];
      }
    } else {
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        if (b * 32 >= T * d.k) break;
        const int e = e_slot[b];
        for (int w = 0; w < n_words; ++w) {
          const uint32_t m = __reduce_or_sync(0xffffffffu, (e >= 0 && (e >> 5) == w) ? 1u << (e & 31) : 0u);
          if (lane == w) act_word |= m;
        }
      }
    }
    if (d.ns > 0) {     // shared experts are active as soon as one row is computed
      const bool any = __ballot_sync(0xffffffffu, lane < T && c_cls[lane] != TEAM_CLS_SKIP) != 0u;
      for (int sh = 0; sh < d.ns && any; ++sh)
        if (lane == ((d.E + sh) >> 5)) act_word |= 1u << ((d.E + sh) & 31);
    }
    if (d.elo > 0 || d.ehi < d.E) {
      // expert parallelism: only this rank's routed experts [elo, ehi) are computed here
      const int lo = lane * 32, hi = lo + 32;
      uint32_t keep = 0u;
      if (hi > d.elo && lo < d.ehi) {
        const int a0 = max(d.elo, lo) - lo, a1 = min(d.ehi, hi) - lo;       // bits [a0, a1)
        keep = (a1 - a0 == 32) ? 0xffffffffu : (((1u << (a1 - a0)) - 1u) << a0);
      }
      act_word &= keep;
    }
    n_act = __reduce_add_sync(0xffffffffu, __popc(act_word));
  }
  // at most (2048 * 20 + 260) items x 64 groups: the products below stay far inside 64 bits and, for the resident
  // modes (at most 260 experts x 64 groups x a grid of a few hundred), inside 32
  int g_lo, g_hi;
  if (GATHER) {
    const long long n_groups = (long long)(*a.n_items) * NG;
    g_lo = (int)(n_groups * blockIdx.x / gridDim.x);
    g_hi = (int)(n_groups * (blockIdx.x + 1) / gridDim.x);
  } else {
    const unsigned n_groups = (unsigned)(n_act * NG);
    g_lo = (int)(n_groups * blockIdx.x / gridDim.x);
    g_hi = (int)(n_groups * (blockIdx.x + 1u) / gridDim.x);
  }

  // fused step: what the selection still owes once the activated set is known -- the second routing round (cold
  // rows inside E_A), the softmax denominators and routing weights, and CTA 0's exports.  Run once per CTA by
  // warps 0 .. T-1, in the shadow of the first weight copies' latency (or after the loop if this CTA has no
  // group at all); the routing weights are first read after the barrier that ends phase 1.
  bool late_done = false;
  auto late_select = [&]() {
    if constexpr (FUSED) {
      if (warp < T) {
        const int t = warp, k = d.k, E = d.E;
        const bool exporter = blockIdx.x == 0;
        float row_max = 0.f, denom = 1.f, w = 0.f;
        if (f_mycls == TEAM_CLS_COLD) {
          const int gs = f_gslot[t];
#pragma unroll
          for (int i = 0; i < kMaxPerLane; ++i)
            if (!((f_mask[gs * 8 + i] >> lane) & 1u)) f_key[i] = kKeyNegInf;      // outside E_A: no candidate
          sort_lane_keys(f_key, f_slot);
          const int n = warp_topk_picks(f_key, f_slot, k, lane,
                                        [&](int j, int e, uint32_t key) {
                                          f_idx[t * k + j] = e;
                                          f_wt[t * k + j] = key_float(key);
                                        },
                                        f_margin);
          if (n < k) {
            if (lane >= n && lane < k) f_idx[t * k + lane] = -1;
            if (exporter && lane == 0) set_status(a.status, TEAM_ERR_STATE, 3);
          }
        }
        __syncwarp();
        if (f_mycls != TEAM_CLS_SKIP) {
          float m = kNegInf;
#pragma unroll
          for (int i = 0; i < kMaxPerLane; ++i) m = fmaxf(m, f_val[i]);
          row_max = warp_max(m);
          float se = 0.f;
#pragma unroll
          for (int i = 0; i < kMaxPerLane; ++i)
            if (i * 32 + lane < E) se += expf(f_val[i] - row_max);
          denom = warp_sum(se);
          TopkResult tr;
          tr.idx = lane < k ? f_idx[t * k + lane] : -1;
          tr.val = lane < k ? f_wt[t * k + lane] : kNegInf;
          tr.margin = f_margin;
          tr.top = row_max;
          w = routing_weight(tr, k, lane, row_max, denom, a.p.norm_topk);
          if (tr.idx < 0) w = 0.f;
          __syncwarp();
          if (lane < k) f_wt[t * k + lane] = w;
        }
        if (exporter) {
          if (lane < k) {
            const int e = f_idx[t * k + lane];
            a.r.topk_idx[t * k + lane] = e;
            a.r.topk_w[t * k + lane] = w;
            if (a.ex.topk_idx) a.ex.topk_idx[t * k + lane] = e;
            if (a.ex.topk_w) a.ex.topk_w[t * k + lane] = w;
          }
          if (lane == 0) {
            a.r.margin[t] = f_margin;
            if (a.ex.margin) a.ex.margin[t] = f_margin;
            a.r.tok_class[t] = (uint8_t)f_mycls;
            if (a.ex.tok_class) a.ex.tok_class[t] = (uint8_t)f_mycls;
          }
          if (a.ex.probs) {
#pragma unroll
            for (int i = 0; i < kMaxPerLane; ++i) {
              const int e = i * 32 + lane;
              if (e < E) a.ex.probs[(size_t)t * E + e] = f_mycls != TEAM_CLS_SKIP ? expf(f_val[i] - row_max) / denom : 0.f;
            }
          }
          // E_A of the groups that are present: written by the group's first row
          const int n_words64 = (E + 63) / 64;
          const int g = min(max(__shfl_sync(0xffffffffu, f_group, t), 0), d.G - 1);
          if (f_gslot[t] == t && lane < n_words64) {
            const uint64_t mk = (uint64_t)f_mask[t * 8 + 2 * lane] | ((uint64_t)f_mask[t * 8 + 2 * lane + 1] << 32);
            a.r.group_mask[(size_t)g * n_words64 + lane] = mk;
            if (a.ex.group_mask) a.ex.group_mask[(size_t)g * n_words64 + lane] = mk;
          }
        }
      }
    }
  };

  int cur_item = -1;
  for (int s_lo = g_lo, s_hi; s_lo < g_hi; s_lo = s_hi) {
    s_hi = min(g_hi, s_lo + PASS);
    const int item0 = s_lo / NG;
    if (GATHER) s_hi = min(s_hi, (item0 + 1) * NG);      // a pass stays inside one work item
    const int ng = s_hi - s_lo;
    // ---- group table: lane q holds item, expert and position of group q ----
    int my_item = -1, my_e = 0, my_gi = 0;
    if (lane < ng) {
      const int grp = s_lo + lane;
      my_item = grp / NG;
      my_gi = grp - my_item * NG;
      if (GATHER) my_e = a.items[my_item].e;
    }
    if (!GATHER) {
      int left = my_item;                   // the my_item-th set bit of the activated set (-1: no group in this lane)
      for (int w = 0; w < n_words; ++w) {
        const uint32_t m = __shfl_sync(0xffffffffu, act_word, w);
        const int c = __popc(m);
        if (left >= 0 && left < c) my_e = w * 32 + st_nth_set_bit(m, left);
        left = left >= c ? left - c : -1;
      }
    }
    // ---- routing weights of the pass's experts, per group and token (read in phase 2, after the barriers):
    //      warp q < ng looks group q's expert up in the rows' choices ----
    auto pass_weights = [&]() {
      const int item = __shfl_sync(0xffffffffu, my_item, warp), e = __shfl_sync(0xffffffffu, my_e, warp);
      if (lane == 0) s_item[warp] = item;
      if (lane < kStRows) {
        float wt = 0.f;
        if (lane < T) {
          if (e >= d.E) {
            wt = c_cls[lane] != TEAM_CLS_SKIP ? 1.f : 0.f;      // a shared expert: every computed row, weight 1
          } else {
            // all loads are independent of each other (no branch between them)
            for (int j = 0; j < d.k; ++j) {
              const int ej = c_idx[lane * d.k + j];
              const float wj = c_wt[lane * d.k + j];
              wt = ej == e ? wj : wt;
            }
          }
        }
        s_w[warp][lane] = wt;
      }
    };
    // ---- issue side: phase-1 chunks, then phase-2 chunks, then empty groups ----
    const int n1 = ng * NCH, n2 = ng * CPG;
    int n_issued = 0, iq = 0, icc = 0;
    const __nv_bfloat16* i_src = nullptr;
    auto issue_one = [&]() {
      const uint32_t dst = ring + (uint32_t)(n_issued % SLOTS) * kStChunkBytes;
      if (n_issued < n1) {
        if (icc == 0) {
          const int e = __shfl_sync(0xffffffffu, my_e, iq), gi = __shfl_sync(0xffffffffu, my_gi, iq);
          i_src = wmat + ((size_t)e * I + gi * 16 + cp_row) * H + ks * KS + cp_piece * 8;
        }
        const __nv_bfloat16* p = i_src + icc * 64;
        st_cp16(dst + cp_off0, p, pol);
        st_cp16(dst + cp_off1, p + 4 * (size_t)H, pol);
        st_cp16(dst + cp_off0 + 1024, p + 8 * (size_t)H, pol);
        st_cp16(dst + cp_off1 + 1024, p + 12 * (size_t)H, pol);
        if (++icc == NCH) {
          icc = 0;
          if (++iq == ng) iq = 0;      // phase 2 walks the groups again
        }
      } else if (n_issued < n1 + n2) {
        // phase 2 walks (row chunk, group): all groups of the pass for the warp's first 64 output rows, then
        // for the next 64, so that the accumulators cover 64 rows at a time
        const int e = __shfl_sync(0xffffffffu, my_e, iq), gi = __shfl_sync(0xffffffffu, my_gi, iq);
        const __nv_bfloat16* p = a.w_down + (((size_t)e * NG + gi) * H + warp * HW) * 16 + lane * 8 + icc * 1024;
        st_cp16(dst + cq_off, p, pol);
        st_cp16(dst + cq_off + 512, p + 256, pol);
        st_cp16(dst + cq_off + 1024, p + 512, pol);
        st_cp16(dst + cq_off + 1536, p + 768, pol);
        if (++iq == ng) {
          iq = 0;
          ++icc;
        }
      }
      st_commit();
      ++n_issued;
    };
#pragma unroll
    for (int b = 0; b < SLOTS - 1; ++b) issue_one();

    if (GATHER) {
      // ---- a new work item: its rows and weights, then its token rows into shared memory (the first weight
      //      chunks are already on their way) ----
      if (warp == 0 && lane < ng) s_item[lane] = item0;
      if (item0 != cur_item) {
        if (warp == 0 && lane < TOK) {
          const WorkItem it = a.items[item0];
          int row = -1;
          float wt = 0.f;
          if (lane < it.n) slot_row_weight(a.perm[it.begin + lane], T, d.k, a.topk_w, row, wt);
          s_row[lane] = row;
          s_wt[lane] = wt;
        }
        __syncthreads();
        for (int idx = tid; idx < TOK * per_row; idx += kStThreads) {
          const int n = idx / per_row, ci = idx - n * per_row;
          const int row = s_row[n];
          uint4 v = make_uint4(0u, 0u, 0u, 0u);
          if (row >= 0) v = st_ldg_stream(a.x + (size_t)row * H + ci * 8);
          *reinterpret_cast<uint4*>(xs + (size_t)n * H * 2 + ((ci ^ (n & 7)) << 4)) = v;
        }
        __syncthreads();
        cur_item = item0;
      }
    } else if (!FUSED && warp < ng) {
      pass_weights();
    }
    if (FUSED && !late_done) {
      late_select();
      late_done = true;
    }

    // ---- phase 1 ----
    int t = 0;     // chunks consumed in this pass
    {
      float acc[NTL][4];
#pragma unroll
      for (int nt = 0; nt < NTL; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
      int q = 0, cc = 0;
      for (; t < n1; ++t) {
        issue_one();
        st_wait_group<SLOTS - 1>();
        __syncwarp();
        const uint32_t slot = ring + (uint32_t)(t % SLOTS) * kStChunkBytes;
        const int p0 = (ks * KS + cc * 64) >> 3;               // first 16-byte piece of the token rows
        uint32_t bf0[NTL][4], bf1[NTL][4];
#pragma unroll
        for (int nt = 0; nt < NTL; ++nt) {
          const uint32_t xrow = xs_lane + (uint32_t)nt * 8 * H * 2;      // token nt * 8 + b_tok: same swizzle
          st_ldmatrix4(xrow + (uint32_t)((p0 + (b_m ^ b_tok)) << 4), bf0[nt]);
          st_ldmatrix4(xrow + (uint32_t)((p0 + ((4 + b_m) ^ b_tok)) << 4), bf1[nt]);
        }
#pragma unroll
        for (int ks16 = 0; ks16 < 4; ++ks16) {
          uint32_t af[4];
          st_ldmatrix4(slot + a1_base + (uint32_t)(((2 * ks16 + a_hi) ^ a1_swz) << 4), af);
#pragma unroll
          for (int nt = 0; nt < NTL; ++nt) {
            const uint32_t* bf = ks16 < 2 ? bf0[nt] : bf1[nt];
            st_mma(acc[nt], af, bf[(ks16 & 1) * 2], bf[(ks16 & 1) * 2 + 1]);
          }
        }
        __syncwarp();                                           // the slot may be overwritten from here on
        if (++cc == NCH) {
          float* r = red + ((size_t)((q * kStSlices + ks) * 2 + tile) * 16) * TOK;
#pragma unroll
          for (int nt = 0; nt < NTL; ++nt) {
            *reinterpret_cast<float2*>(r + g * TOK + nt * 8 + 2 * c) = make_float2(acc[nt][0], acc[nt][1]);
            *reinterpret_cast<float2*>(r + (g + 8) * TOK + nt * 8 + 2 * c) = make_float2(acc[nt][2], acc[nt][3]);
            acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
          }
          cc = 0;
          ++q;
        }
      }
    }
    __syncthreads();
    if (FUSED && warp < ng) pass_weights();      // the routing weights are complete by now (late selection)
    // ---- sum the slices, SwiGLU ----
    for (int idx = tid; idx < ng * 16 * TOK; idx += kStThreads) {
      const int qq = idx / (16 * TOK), r = (idx / TOK) & 15, n = idx % TOK;
      float gs = 0.f, us = 0.f;
#pragma unroll
      for (int s = 0; s < kStSlices; ++s) {
        const float* base = red + ((size_t)((qq * kStSlices + s) * 2) * 16) * TOK + r * TOK + n;
        gs += base[0];
        us += base[16 * TOK];
      }
      s_act[(qq * TOK + n) * 16 + r] = __float2bfloat16_rn(gs / (1.f + expf(-gs)) * us);     // unused token columns are zero (x is)
    }
    __syncthreads();
    // ---- phase 2: for each 64-row chunk of this warp's output rows, all groups of the pass ----
#pragma unroll 1
    for (int ch = 0; ch < CPG; ++ch) {
      float acc[4][NTL][4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int nt = 0; nt < NTL; ++nt) acc[u][nt][0] = acc[u][nt][1] = acc[u][nt][2] = acc[u][nt][3] = 0.f;
      for (int q = 0; q < ng; ++q, ++t) {
        issue_one();
        st_wait_group<SLOTS - 1>();
        __syncwarp();
        const uint32_t slot = ring + (uint32_t)(t % SLOTS) * kStChunkBytes;
        uint32_t b0[NTL], b1[NTL];
#pragma unroll
        for (int nt = 0; nt < NTL; ++nt) {
          const __nv_bfloat16* ar = s_act + (q * TOK + nt * 8 + g) * 16;
          b0[nt] = *reinterpret_cast<const uint32_t*>(ar + 2 * c);
          b1[nt] = *reinterpret_cast<const uint32_t*>(ar + 8 + 2 * c);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          uint32_t af[4];
          st_ldmatrix4(slot + u * 512 + a2_off, af);
#pragma unroll
          for (int nt = 0; nt < NTL; ++nt) st_mma(acc[u][nt], af, b0[nt], b1[nt]);
        }
        __syncwarp();
        // the expert's groups in this pass are summed: scale by the routing weights and add to y
        if (q == ng - 1 || s_item[q + 1] != s_item[q]) {
          // ordered combine (one-kernel step only): the CTA's own partial output, every element owned by one thread,
          // summed over the CTAs in index order at the end of the kernel; otherwise fp32 reductions into y
          const bool ordered = FUSED && a.ordered != nullptr;
          float* y0 = (ordered ? a.ordered + (size_t)blockIdx.x * T * H : a.y) + warp * HW + ch * 64 + g;
#pragma unroll
          for (int nt = 0; nt < NTL; ++nt) {
            const int cA = nt * 8 + 2 * c, cB = cA + 1;          // this thread's two token columns
            const float wA = GATHER ? s_wt[cA] : s_w[q][cA], wB = GATHER ? s_wt[cB] : s_w[q][cB];
            const int rA = GATHER ? s_row[cA] : cA, rB = GATHER ? s_row[cB] : cB;
            float* yA = y0 + (size_t)max(rA, 0) * H;
            float* yB = y0 + (size_t)max(rB, 0) * H;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              if (ordered) {
                if (wA != 0.f) {
                  yA[u * 16] += wA * acc[u][nt][0];
                  yA[u * 16 + 8] += wA * acc[u][nt][2];
                }
                if (wB != 0.f) {
                  yB[u * 16] += wB * acc[u][nt][1];
                  yB[u * 16 + 8] += wB * acc[u][nt][3];
                }
              } else {
                if (wA != 0.f) {
                  atomicAdd(yA + u * 16, wA * acc[u][nt][0]);
                  atomicAdd(yA + u * 16 + 8, wA * acc[u][nt][2]);
                }
                if (wB != 0.f) {
                  atomicAdd(yB + u * 16, wB * acc[u][nt][1]);
                  atomicAdd(yB + u * 16 + 8, wB * acc[u][nt][3]);
                }
              }
              acc[u][nt][0] = acc[u][nt][1] = acc[u][nt][2] = acc[u][nt][3] = 0.f;
            }
          }
        }
      }
    }
    st_wait_group<0>();     // only empty groups can be pending here
    __syncthreads();        // s_act, s_w and the partial sums are free for the next pass
  }
  if (FUSED && !late_done) late_select();      // a CTA without any group still owes its part (CTA 0: the exports)
  if constexpr (FUSED) {
    if (a.ordered != nullptr) {
      // ---- ordered combine: a second grid barrier, then y = sum over the CTAs' partial outputs in index order ----
      __syncthreads();
      if (tid == 0) {
        __threadfence();
        atomicAdd(a.arrivals, 1ull);
        const unsigned long long target = bar_target - (unsigned long long)a.extra_arrivals + gridDim.x;
        const long long t_begin = clock64();
        while (st_ld_acquire(a.arrivals) < target) {
          if (clock64() - t_begin > a.spin_cycles) {
            *f_flag = 1;
            break;
          }
        }
      }
      __syncthreads();
      if (*f_flag) {
        if (tid == 0) set_status(a.status, TEAM_ERR_TIMEOUT, 21);
        return;
      }
      const int total4 = T * H / 4, n_cta = gridDim.x;
      for (int i = blockIdx.x * kStThreads + tid; i < total4; i += n_cta * kStThreads) {
        const int t = (i * 4) / H;
        if (c_cls[t] == TEAM_CLS_SKIP) continue;
        float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int cta = 0; cta < n_cta; ++cta) {
          const float4 v = __ldcg(reinterpret_cast<const float4*>(a.ordered + (size_t)cta * T * H) + i);
          sum.x += v.x; sum.y += v.y; sum.z += v.z; sum.w += v.w;
        }
        reinterpret_cast<float4*>(a.y)[i] = sum;
      }
    }
  }
}

// Few rows: all rows resident.  Up to kStGatherMaxRows rows: work items whose rows are gathered per item, of
// 8 token-slots up to kStOneTileMaxRows rows per call (few experts see more than 8 rows there) and of 16 above
// (an expert with more slots than an item holds is streamed once per item, which beyond kStGatherMaxRows costs
// more than the tensor-memory kernel's larger tiles).
constexpr int kStGatherMaxRows = TEAM_MAX_ROWS;
constexpr int kStOneTileMaxRows = 64;
bool experts_stream_supported(int max_rows, int hidden, int inter) {
  return max_rows <= kStGatherMaxRows && (hidden == 1024 || hidden == 2048) && inter % 16 == 0;
}
bool experts_stream_gathers(int max_rows) { return max_rows > kStRows; }
static int stream_token_tiles(int max_rows) { return max_rows > kStOneTileMaxRows ? 2 : 1; }
int experts_stream_item_tile(int max_rows) { return kStRows * stream_token_tiles(max_rows); }

static const void* stream_kernel(int hidden, int max_rows) {
  const bool gather = experts_stream_gathers(max_rows), two = stream_token_tiles(max_rows) == 2;
  if (hidden == 1024) {
    if (!gather) return reinterpret_cast<const void*>(&k_experts_stream<1, false, 1>);
    return two ? reinterpret_cast<const void*>(&k_experts_stream<1, true, 2>) : reinterpret_cast<const void*>(&k_experts_stream<1, true, 1>);
  }
  if (!gather) return reinterpret_cast<const void*>(&k_experts_stream<2, false, 1>);
  return two ? reinterpret_cast<const void*>(&k_experts_stream<2, true, 2>) : reinterpret_cast<const void*>(&k_experts_stream<2, true, 1>);
}

static const void* fused_kernel(int hidden) {
  return hidden == 1024 ? reinterpret_cast<const void*>(&k_experts_stream<1, false, 1, true>)
                        : reinterpret_cast<const void*>(&k_experts_stream<2, false, 1, true>);
}

cudaError_t configure_experts_stream(int hidden, int max_rows) {
  const void* fn = stream_kernel(hidden, max_rows);
  cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)stream_smem_bytes(hidden, stream_token_tiles(max_rows)));
  if (e == cudaSuccess) e = cudaFuncSetAttribute(fn, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
  if (e == cudaSuccess && !experts_stream_gathers(max_rows)) {
    fn = fused_kernel(hidden);
    e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)stream_smem_bytes(hidden, 1, true));
    if (e == cudaSuccess) e = cudaFuncSetAttribute(fn, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
  }
  return e;
}

// The fused step can run when every CTA of the grid is resident at once (they meet at a barrier): one CTA per
// SM fits by construction (launch bounds and shared memory allow exactly one), the occupancy query confirms it.
bool step_fused_supported(int hidden, int max_rows, int n_experts, int grid) {
  if (experts_stream_gathers(max_rows) || !(hidden == 1024 || hidden == 2048) || n_experts > TEAM_MAX_EXPERTS) return false;
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fused_kernel(hidden), kStThreads,
                                                    stream_smem_bytes(hidden, 1, true)) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  return per_sm >= 1 && grid <= per_sm * sms;
}

cudaError_t launch_step_fused(const void* x, const float* w_router, const void* w_gate, const void* w_up, const void* w_down,
                              StepPtrs st, Workspace ws, RoutePtrs ex, float* y, Dims d, Policy p, int grid,
                              long long spin_cycles, int extra_arrivals, float* ordered, cudaStream_t s) {
  StArgs a = {};
  a.ordered = ordered;
  a.x = static_cast<const __nv_bfloat16*>(x);
  a.w_gate = static_cast<const __nv_bfloat16*>(w_gate);
  a.w_up = static_cast<const __nv_bfloat16*>(w_up);
  a.w_down = static_cast<const __nv_bfloat16*>(w_down);
  a.y = y;
  a.d = d;
  a.w_router = w_router;
  a.logits = ws.logits;
  a.st = st;
  a.p = p;
  a.r = ws.r;
  a.ex = ex;
  a.arrivals = ws.arrivals;
  a.status = ws.status;
  a.spin_cycles = spin_cycles;
  a.extra_arrivals = extra_arrivals;
  // Cooperative: all CTAs are resident together, so the barrier's wait ends.  Programmatic serialization: the
  // launch latency and the first router weight loads hide behind the tail of the preceding kernel.
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kStThreads);
  cfg.dynamicSmemBytes = stream_smem_bytes(d.H, 1, true);
  cfg.stream = s;
  cudaLaunchAttribute attrs[2];
  attrs[0].id = cudaLaunchAttributeCooperative;
  attrs[0].val.cooperative = 1;
  attrs[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attrs[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attrs;
  cfg.numAttrs = 2;
  void* params[1] = {&a};
  return cudaLaunchKernelExC(&cfg, fused_kernel(d.H), params);
}

cudaError_t launch_experts_stream(const void* x, const void* w_gate, const void* w_up, const void* w_down, Workspace ws,
                                  float* y, Dims d, int max_rows, int grid, cudaStream_t s) {
  StArgs a = {};
  a.x = static_cast<const __nv_bfloat16*>(x);
  a.w_gate = static_cast<const __nv_bfloat16*>(w_gate);
  a.w_up = static_cast<const __nv_bfloat16*>(w_up);
  a.w_down = static_cast<const __nv_bfloat16*>(w_down);
  a.perm = ws.r.perm;
  a.topk_idx = ws.r.topk_idx;
  a.tok_class = ws.r.tok_class;
  a.topk_w = ws.r.topk_w;
  a.items = ws.items;
  a.n_items = ws.n_items;
  a.y = y;
  a.d = d;
  // Programmatic serialization: staging the token rows overlaps the selection kernel.
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kStThreads);
  cfg.dynamicSmemBytes = stream_smem_bytes(d.H, stream_token_tiles(max_rows));
  cfg.stream = s;
  cudaLaunchAttribute attrs[1];
  attrs[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attrs[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attrs;
  cfg.numAttrs = 1;
  void* params[1] = {&a};
  return cudaLaunchKernelExC(&cfg, stream_kernel(d.H, max_rows), params);
}

}  // namespace team
