// Expert kernel for the few-rows regime (T <= 8 rows, bf16 weights): a weight-streaming kernel.
//
// With a handful of rows the SwiGLU experts are a matrix-vector problem: ~1 MB of weights per SM and
// a few hundred kFLOP.  Staging tiles for the tensor-memory path costs more in hand-offs between
// warps than the math is worth, so here every warp is its own pipeline: it copies 2 KB chunks of
// weights (16 rows x 128 bytes) from HBM into a private ring in shared memory with asynchronous
// copies, several chunks ahead, and multiplies each chunk with the token rows using warp-level mma
// (m16n8k16: 16 weight rows x 8 tokens).  No warp ever waits for another one inside a phase; one
// block-wide barrier per pass separates the gate/up phase from the down phase.
//
// The work partition is the expert kernel's: the intermediate dimension of every activated expert is
// cut into groups of 16 columns; a group costs 16 gate rows + 16 up rows of W (phase 1) and a quarter
// of the W_down tiles of its 64-column window (phase 2); the global list of groups is cut into one
// contiguous range per CTA.  Windows cut by a range boundary are shared by neighbouring CTAs through
// the activation scratch in global memory and one counter per window (cooperative launch, bounded
// waits; a CTA's head window comes last when its range spans several passes, so waits cannot form a
// cycle).
//
//   phase 1   warp = (gate | up tile of 16 rows) x (one of 8 slices of the hidden dimension), for every
//             group of the pass in turn; partial sums of a slice go to shared memory.
//   barrier   sum the 8 slices, a = silu(gate) * up, round to bf16, publish to the scratch, count.
//   phase 2   per window and owned tile range: warps take 16-row units of W_down (128 bytes per row),
//             read the window's activations from the scratch (L2), scale by the routing weight and
//             add into y with fp32 reductions.  Fully owned windows go first, shared ones after, so
//             that the neighbours' activations have arrived by the time they are needed.
//
// A warp's copies run ahead across the barrier: while the slices are being summed, the first W_down
// units of phase 2 are already on their way.
#include "team_common.cuh"

namespace team {

constexpr int kStThreads = 512;
constexpr int kStWarps = 16;
constexpr int kStSlices = 8;                    // slices of the hidden dimension in phase 1
constexpr int kStRows = 8;                      // token rows (n of the mma)
constexpr int kStScWindows = 2;                 // windows per pass
constexpr int kStScGroups = kStScWindows * 4;   // groups whose partial sums fit in shared memory
constexpr int kStChunkBytes = 2048;             // 16 rows x 128 bytes
constexpr int kStRedBytes = kStScGroups * kStSlices * 2 * 16 * kStRows * 4;
constexpr unsigned long long kStWaitCycles = 2000000000ull;   // ~1 s

struct StArgs {
  const __nv_bfloat16* x;       // [T, H]
  const __nv_bfloat16* w_gate;  // [E + ns, I, H]
  const __nv_bfloat16* w_up;
  const __nv_bfloat16* w_down;  // [E + ns, H, I]
  const int32_t* perm;
  const float* topk_w;
  const WorkItem* items;
  const int32_t* n_items;
  __nv_bfloat16* act_g;         // [items][16][I]
  int32_t* win_flags;           // [items * I/64]
  float* y;                     // [T, H]
  int32_t* status;
  Dims d;
};

__device__ __forceinline__ uint32_t st_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void st_cp16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
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
__device__ __forceinline__ uint32_t st_ldg_l2(const void* p) {      // data written by other CTAs during this launch
  uint32_t v;
  asm volatile("ld.global.cg.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ int st_ld_acquire(const int32_t* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
// d += A(16x16, rows g / g+8) * B(16x8), bf16 inputs, fp32 accumulate
__device__ __forceinline__ void st_mma(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// shared memory: token rows | partial sums [group][slice][gate, up][16 rows][8 tokens] | per-warp rings
__host__ __device__ inline int stream_ring_slots(int H) { return H <= 2048 ? 4 : 3; }
__host__ __device__ inline size_t stream_smem_bytes(int H) {
  return (size_t)kStRows * H * 2 + kStRedBytes + (size_t)kStWarps * stream_ring_slots(H) * kStChunkBytes;
}

// Phase-2 job: the CTA's groups [a, b) of window W (global window index) own the W_down row tiles
// [a*HT/4, b*HT/4) of that window; a 16-row unit of them is what one warp handles at a time.
struct StJob {
  int W, a, b;
};

template <int SLOTS>
__global__ void __launch_bounds__(kStThreads, 1) k_experts_stream(StArgs a) {
  extern __shared__ __align__(128) unsigned char st_smem[];
  __shared__ int s_item[kStScGroups], s_col[kStScGroups];
  const Dims d = a.d;
  const int H = d.H, I = d.I, T = d.T;
  unsigned char* xs = st_smem;                                                    // [8][H] bf16, 16-byte pieces swizzled
  float* red = reinterpret_cast<float*>(st_smem + (size_t)kStRows * H * 2);      // [group][slice][2][16][8]
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, c = lane & 3;        // fragment row (and token of the B fragment), k / token pair
  const int NG = I / 16, WPI = NG / 4, HT = H / 128;
  const int KS = H / kStSlices, NCH = KS / 64;  // elements per slice, 64-wide chunks per slice

  // ---- token rows into shared memory (an input of the call: may overlap the selection kernel) ----
  {
    const int per_row = H / 8;
    for (int idx = tid; idx < kStRows * per_row; idx += kStThreads) {
      const int n = idx / per_row, ci = idx - n * per_row;
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (n < T) v = st_ldg_stream(a.x + (size_t)n * H + ci * 8);
      *reinterpret_cast<uint4*>(xs + (size_t)n * H * 2 + ((ci ^ n) << 4)) = v;
    }
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");     // the selection kernel's tables are complete from here on
  __syncthreads();

  const long long n_groups = (long long)(*a.n_items) * NG;
  const int g_lo = (int)(n_groups * blockIdx.x / gridDim.x), g_hi = (int)(n_groups * (blockIdx.x + 1) / gridDim.x);
  const bool multi = g_hi > (((g_lo >> 2) + kStScWindows) << 2);   // more than one pass
  bool ok = true;

  // ---- this warp's ring and its fixed lane roles ----
  const uint32_t ring = st_smem_u32(st_smem + (size_t)kStRows * H * 2 + kStRedBytes + (size_t)warp * SLOTS * kStChunkBytes);
  const int cp_row = lane >> 3, cp_piece = lane & 7;                 // copies: rows cp_row + 4j, one 16-byte piece
  const uint32_t cp_off0 = cp_row * 128 + ((cp_piece ^ cp_row) << 4);          // rows cp_row, cp_row + 8 (+1024)
  const uint32_t cp_off1 = (cp_row + 4) * 128 + ((cp_piece ^ (cp_row + 4)) << 4);
  const int a_row = (lane & 7) + ((lane >> 3) & 1) * 8, a_hi = lane >> 4;      // ldmatrix: A tile row, low / high k half
  const uint32_t a_base = a_row * 128;
  const int a_swz = a_row & 7;
  const int b_tok = lane & 7, b_m = lane >> 3;                                 // ldmatrix: token row, k piece
  const uint32_t xs_lane = st_smem_u32(xs) + (uint32_t)b_tok * H * 2;
  const int tile = warp & 1, ks = warp >> 1;     // phase 1: this warp's 16-row tile (gate | up) and hidden slice
  const __nv_bfloat16* wmat = tile ? a.w_up : a.w_gate;

  // One pass: phase 1 over groups [s_lo, s_hi) (may be empty), then the phase-2 jobs.
  auto run_pass = [&](int s_lo, int s_hi, const StJob* jobs, int nj) {
    const int ng = s_hi - s_lo;
    // ---- group table: lane q holds expert and first column of group q ----
    int my_e = 0, my_col = 0;
    if (lane < ng) {
      const int grp = s_lo + lane;
      const int item = grp / NG;
      my_e = a.items[item].e;
      my_col = (grp - item * NG) * 16;
      if (warp == 0) {
        s_item[lane] = item;
        s_col[lane] = my_col;
      }
    }
    // ---- job table: expert of each phase-2 job ----
    int je[kStScWindows] = {};
#pragma unroll
    for (int jj = 0; jj < kStScWindows; ++jj)
      if (jj < nj) je[jj] = a.items[(4 * jobs[jj].W) / NG].e;
    const int n1 = ng * NCH;
    // ---- issue side: phase-1 chunks, then phase-2 units, then empty groups ----
    auto n_units = [&](int jj) { const StJob& j = jobs[jj]; return (j.b * HT / 4 - j.a * HT / 4) * 8; };
    auto first_valid = [&](int& jj, int& u) {
      while (jj < nj && u >= n_units(jj)) { ++jj; u = warp; }
    };
    int n_issued = 0, iq = 0, icc = 0;
    const __nv_bfloat16* p1_src = nullptr;
    int ij = 0, iu = warp;
    first_valid(ij, iu);
    auto issue_one = [&]() {
      const uint32_t dst = ring + (uint32_t)(n_issued % SLOTS) * kStChunkBytes;
      const __nv_bfloat16* src = nullptr;
      size_t stride = 0;
      if (n_issued < n1) {
        if (icc == 0) {
          const int e = __shfl_sync(0xffffffffu, my_e, iq), col = __shfl_sync(0xffffffffu, my_col, iq);
          p1_src = wmat + ((size_t)e * I + col) * H + (size_t)ks * KS;
        }
        src = p1_src + icc * 64;
        stride = H;
        if (++icc == NCH) { icc = 0; ++iq; }
      } else if (ij < nj) {
        const StJob& j = jobs[ij];
        const int item = (4 * j.W) / NG, w = j.W - item * WPI;
        int e = je[0];
#pragma unroll
        for (int jj = 1; jj < kStScWindows; ++jj)
          if (jj == ij) e = je[jj];
        const int h0 = (j.a * HT / 4) * 128 + iu * 16;
        src = a.w_down + ((size_t)e * H + h0) * I + w * 64;
        stride = I;
        iu += kStWarps;
        first_valid(ij, iu);
      }
      if (src != nullptr) {
        const __nv_bfloat16* p = src + (size_t)cp_row * stride + cp_piece * 8;
        st_cp16(dst + cp_off0, p);
        st_cp16(dst + cp_off1, p + 4 * stride);
        st_cp16(dst + cp_off0 + 1024, p + 8 * stride);
        st_cp16(dst + cp_off1 + 1024, p + 12 * stride);
      }
      st_commit();
      ++n_issued;
    };
    // A fragments of k16 step s of the chunk in a slot
    auto load_a = [&](uint32_t slot, int s, uint32_t (&af)[4]) {
      st_ldmatrix4(slot + a_base + (uint32_t)(((2 * s + a_hi) ^ a_swz) << 4), af);
    };
#pragma unroll
    for (int b = 0; b < SLOTS - 1; ++b) issue_one();
    // ---- routing weights of this thread's two tokens (2c, 2c + 1) for each job's expert ----
    float jwA[kStScWindows] = {}, jwB[kStScWindows] = {};
#pragma unroll
    for (int jj = 0; jj < kStScWindows; ++jj) {
      if (jj < nj) {
        const WorkItem it = a.items[(4 * jobs[jj].W) / NG];
        int row = -1;
        float wt = 0.f;
        if (lane < it.n) slot_row_weight(a.perm[it.begin + lane], T, d.k, a.topk_w, row, wt);
#pragma unroll
        for (int r = 0; r < kStRows; ++r) {
          const int rr = __shfl_sync(0xffffffffu, row, r);
          const float ww = __shfl_sync(0xffffffffu, wt, r);
          if (rr == 2 * c) jwA[jj] = ww;
          if (rr == 2 * c + 1) jwB[jj] = ww;
        }
      }
    }
    int t = 0;     // chunks consumed in this pass
    if (ng > 0) {
      // ---- phase 1 ----
      float acc[4] = {0.f, 0.f, 0.f, 0.f};
      int q = 0, cc = 0;
      for (; t < n1; ++t) {
        issue_one();
        st_wait_group<SLOTS - 1>();
        __syncwarp();
        const uint32_t slot = ring + (uint32_t)(t % SLOTS) * kStChunkBytes;
        const int p0 = (ks * KS + cc * 64) >> 3;               // first 16-byte piece of the token rows
        uint32_t bf0[4], bf1[4];
        st_ldmatrix4(xs_lane + (uint32_t)((p0 + (b_m ^ b_tok)) << 4), bf0);
        st_ldmatrix4(xs_lane + (uint32_t)((p0 + ((4 + b_m) ^ b_tok)) << 4), bf1);
        uint32_t af[4];
        load_a(slot, 0, af);
        st_mma(acc, af, bf0[0], bf0[1]);
        load_a(slot, 1, af);
        st_mma(acc, af, bf0[2], bf0[3]);
        load_a(slot, 2, af);
        st_mma(acc, af, bf1[0], bf1[1]);
        load_a(slot, 3, af);
        st_mma(acc, af, bf1[2], bf1[3]);
        __syncwarp();                                           // the slot may be overwritten from here on
        if (++cc == NCH) {
          float* r = red + ((size_t)((q * kStSlices + ks) * 2 + tile) * 16) * kStRows;
          *reinterpret_cast<float2*>(r + g * kStRows + 2 * c) = make_float2(acc[0], acc[1]);
          *reinterpret_cast<float2*>(r + (g + 8) * kStRows + 2 * c) = make_float2(acc[2], acc[3]);
          acc[0] = acc[1] = acc[2] = acc[3] = 0.f;
          cc = 0;
          ++q;
        }
      }
      __syncthreads();
      // ---- sum the slices, SwiGLU, publish ----
      for (int idx = tid; idx < ng * 16 * kStRows; idx += kStThreads) {
        const int qq = idx >> 7, r = (idx >> 3) & 15, n = idx & 7;
        float gs = 0.f, us = 0.f;
#pragma unroll
        for (int s = 0; s < kStSlices; ++s) {
          const float* base = red + ((size_t)((qq * kStSlices + s) * 2) * 16) * kStRows + r * kStRows + n;
          gs += base[0];
          us += base[16 * kStRows];
        }
        if (n < T)
          a.act_g[((size_t)s_item[qq] * 16 + n) * I + s_col[qq] + r] = __float2bfloat16_rn(gs / (1.f + expf(-gs)) * us);
      }
      __syncthreads();
      if (tid < kStScWindows) {
        const int w = (s_lo >> 2) + tid;
        if (w <= ((s_hi - 1) >> 2)) {
          __threadfence();      // the CTA's activations are visible device-wide before the count moves
          atomicAdd(a.win_flags + w, min(s_hi, 4 * w + 4) - max(s_lo, 4 * w));
        }
      }
    }
    // ---- phase 2 ----
    // Activations of a job's window as B fragments, once all four groups are published.  Without
    // `block` a window that is not complete yet is left for later.
    uint32_t bfr[kStScWindows][4][2] = {};
    bool ready[kStScWindows] = {};
    auto prep = [&](int jj, bool block) {
      const StJob& j = jobs[jj];
      bool have = j.a == 0 && j.b == 4;        // all four groups are this CTA's own
      if (!have) {
        int seen = 0;
        if (lane == 0) {
          const unsigned long long t0 = clock64();
          while ((seen = st_ld_acquire(a.win_flags + j.W)) < 4 && block) {
            __nanosleep(64);
            if (clock64() - t0 > kStWaitCycles) {
              set_status(a.status, TEAM_ERR_TIMEOUT, 21);
              break;
            }
          }
        }
        seen = __shfl_sync(0xffffffffu, seen, 0);
        have = seen >= 4;
        if (block && !have) ok = false;
      }
      if (have) {
        const int item = (4 * j.W) / NG, w = j.W - item * WPI;
        const __nv_bfloat16* ap = a.act_g + ((size_t)item * 16 + g) * I + w * 64 + 2 * c;
#pragma unroll
        for (int s = 0; s < 4; ++s) {
          bfr[jj][s][0] = st_ldg_l2(ap + s * 16);
          bfr[jj][s][1] = st_ldg_l2(ap + s * 16 + 8);
        }
        ready[jj] = true;
      }
    };
#pragma unroll
    for (int jj = 0; jj < kStScWindows; ++jj)
      if (jj < nj && ok) prep(jj, false);
    int cj = 0, cu = warp, cur_job = -1;
    first_valid(cj, cu);
    uint32_t cur[4][2] = {};
    float wA = 0.f, wB = 0.f;
    for (; cj < nj; ++t) {
      issue_one();
      st_wait_group<SLOTS - 1>();
      __syncwarp();
      if (cj != cur_job && ok) {
#pragma unroll
        for (int jj = 0; jj < kStScWindows; ++jj) {
          if (jj == cj) {
            if (!ready[jj]) prep(jj, true);
#pragma unroll
            for (int s = 0; s < 4; ++s) {
              cur[s][0] = bfr[jj][s][0];
              cur[s][1] = bfr[jj][s][1];
            }
            wA = jwA[jj];
            wB = jwB[jj];
          }
        }
        cur_job = cj;
      }
      if (ok) {      // after a wait ran out the warp only drains its copies
        const uint32_t slot = ring + (uint32_t)(t % SLOTS) * kStChunkBytes;
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        uint32_t af[4];
#pragma unroll
        for (int s = 0; s < 4; ++s) {
          load_a(slot, s, af);
          st_mma(acc, af, cur[s][0], cur[s][1]);
        }
        const int h = (jobs[cj].a * HT / 4) * 128 + cu * 16 + g;
        float* y0 = a.y + (size_t)(2 * c) * H + h;
        if (wA != 0.f) {
          atomicAdd(y0, wA * acc[0]);
          atomicAdd(y0 + 8, wA * acc[2]);
        }
        if (wB != 0.f) {
          atomicAdd(y0 + H, wB * acc[1]);
          atomicAdd(y0 + H + 8, wB * acc[3]);
        }
      }
      __syncwarp();
      cu += kStWarps;
      first_valid(cj, cu);
    }
    st_wait_group<0>();     // only empty groups can be pending here
    __syncwarp();
  };

  // ---- passes: fully owned windows first, shared ones after; a multi-pass range keeps its head window for last ----
  for (int s_lo = g_lo, s_hi; s_lo < g_hi; s_lo = s_hi) {
    s_hi = min(g_hi, ((s_lo >> 2) + kStScWindows) << 2);
    StJob jobs[kStScWindows];
    int nj = 0;
#pragma unroll
    for (int pass = 0; pass < 2; ++pass) {
#pragma unroll
      for (int k = 0; k < kStScWindows; ++k) {
        const int w = (s_lo >> 2) + k;
        if (w <= ((s_hi - 1) >> 2)) {
          const int ja = max(s_lo, 4 * w) - 4 * w, jb = min(s_hi, 4 * w + 4) - 4 * w;
          const bool full = ja == 0 && jb == 4;
          const bool deferred = multi && w == (g_lo >> 2) && (g_lo & 3) != 0;
          if (full == (pass == 0) && !deferred && ja * HT / 4 < jb * HT / 4) {
            jobs[nj].W = w;
            jobs[nj].a = ja;
            jobs[nj].b = jb;
            ++nj;
          }
        }
      }
    }
    run_pass(s_lo, s_hi, jobs, nj);
  }
  if (multi && (g_lo & 3) != 0) {
    StJob job;
    job.W = g_lo >> 2;
    job.a = g_lo & 3;
    job.b = min(g_hi, 4 * job.W + 4) - 4 * job.W;
    if (job.a * HT / 4 < job.b * HT / 4) run_pass(g_lo, g_lo, &job, 1);
  }
}

bool experts_stream_supported(int max_rows, int hidden, int inter) {
  return max_rows <= kStRows && hidden % (kStSlices * 64) == 0 && hidden <= 4096 && inter % 64 == 0;
}

cudaError_t configure_experts_stream(int hidden) {
  const void* fn = stream_ring_slots(hidden) == 4 ? reinterpret_cast<const void*>(&k_experts_stream<4>)
                                                  : reinterpret_cast<const void*>(&k_experts_stream<3>);
  cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)stream_smem_bytes(stream_ring_slots(hidden) == 4 ? 2048 : 4096));
  if (e == cudaSuccess) e = cudaFuncSetAttribute(fn, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
  return e;
}

cudaError_t launch_experts_stream(const void* x, const void* w_gate, const void* w_up, const void* w_down, Workspace ws,
                                  float* y, Dims d, int grid, cudaStream_t s) {
  StArgs a;
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
  // Cooperative: CTAs that share a window wait for each other's activations, so all must be resident.
  // Programmatic serialization: staging the token rows overlaps the selection kernel.
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kStThreads);
  cfg.dynamicSmemBytes = stream_smem_bytes(d.H);
  cfg.stream = s;
  cudaLaunchAttribute attrs[2];
  attrs[0].id = cudaLaunchAttributeCooperative;
  attrs[0].val.cooperative = 1;
  attrs[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attrs[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attrs;
  cfg.numAttrs = 2;
  return stream_ring_slots(d.H) == 4 ? cudaLaunchKernelEx(&cfg, k_experts_stream<4>, a)
                                     : cudaLaunchKernelEx(&cfg, k_experts_stream<3>, a);
}

}  // namespace team
