// Grouped SwiGLU experts on the tensor cores (tcgen05 / tensor memory) for calls with many rows.
//
// With tens of token-slots per activated expert the SwiGLU experts (Eq. 1) are two grouped GEMMs with the
// weights on the M side (128 rows per instruction) and an expert's token-slots on the N side (up to 128, all
// of them in one pass, so an expert's weights cross HBM once however many rows chose it):
//
//   kernel A   D[128, N] = Wgu_tile[128, H] * X[N, H]^T      128 rows = 64 intermediate columns, stored as four
//              blocks of [16 gate rows | 16 up rows]; SwiGLU straight from tensor memory (a gate row and its up
//              row sit 16 lanes apart in one warp), rounded to bf16, written as the B tiles kernel B reads.
//   kernel B   D[128, N] = Wd_tile[128 hidden rows, I] * A[N, I]^T, scaled by the slot's routing weight and
//              added into y[row, :] with fp32 reductions (a row's k experts meet there).
//
// Both are the same pipeline with a different epilogue.  A unit of work is (chunk, tile): a chunk is a run of
// up to 128 token-slots of one activated expert (a work item of the selection kernel), a tile is 64
// intermediate columns (A) or 128 hidden rows (B).  The global list of units is cut into one contiguous range
// per CTA (grid = number of SMs): every unit of a kernel moves the same weight bytes, no CTA ever waits for
// another one, nothing is exchanged between CTAs inside a kernel.
//
// Operands.  Weights are read from a tile-major copy made once per layer (team_pack_w_tiles): every
// [128 rows x 64 k] bf16 tile is 16 KB contiguous and already in the 128-byte-swizzled K-major layout the
// tensor core reads, so a pipeline stage is two one-dimensional bulk copies (weight tile from HBM with an
// evict-first hint, token tile from L2) that complete on the stage's mbarrier.  The token tiles of kernel A
// are gathered per chunk by a small kernel (k_gather_tiles) into the same layout; those of kernel B are what
// kernel A wrote.
//
// Warp roles (192 threads): warp 0 = producer (one lane issues the bulk copies), warp 1 = MMA issuer and
// owner of the tensor memory (converged warp, one elected lane issues), warps 2-5 = epilogue (one lane
// quarter of the accumulator each).  Two accumulators of 128 columns: the tensor core works on the next unit
// while the epilogue drains the previous one.  Every wait is bounded; on expiry the kernel records
// TEAM_ERR_TIMEOUT, leaves its loops, lets its copies land, frees its tensor memory and returns.
#include "team_common.cuh"
#include "team_tc_ptx.cuh"

namespace team {

constexpr int kTileThreads = 192;
constexpr int kTileBytes = 128 * 128;          // one [128 rows x 64 bf16] tile
constexpr int kTileElems = kTileBytes / 2;
constexpr int kTileStages = 6;                 // pipeline stages: weight tile + token tile each
constexpr int kStageBytes = 2 * kTileBytes;
constexpr int kTileChunk = 128;                // token-slots per chunk at most (N of the MMA)
constexpr int kTmemCols = 256;                 // two accumulators of 128 columns
constexpr int kTileSmemBytes = 1024 + kTileStages * kStageBytes + 4 * kTileChunk * 8 + 256;

enum { kEpiSwiglu = 0, kEpiCombine = 1 };

__host__ __device__ inline int pad16(int n) { return (n + 15) & ~15; }
// First padded row of chunk c in the gathered tables: chunks follow each other in dispatch order, each padded
// to a multiple of 16 rows (at most 15 rows of padding, so 16 rows of slack per chunk keep them apart).
__host__ __device__ inline int chunk_row0(const WorkItem& it, int c) { return it.begin + 16 * c; }

// ---------------------------------------------------------------------------------------------------------
// Weight layout: row-major -> tile-major, pre-swizzled (once per layer)
// ---------------------------------------------------------------------------------------------------------
// gu tiles: [e][u = I/64][kb = H/64][128 rows][64 k]; row r = blk*32 + m*16 + i16 holds (m ? W_up : W_gate)
//           [e][u*64 + blk*16 + i16][kb*64 ...]; 16-byte piece p of row r is stored at piece p ^ (r & 7).
// d tiles:  [e][ht = H/128][kb = I/64][128 rows][64 k]; row r holds W_down[e][ht*128 + r][kb*64 ...].
__global__ void __launch_bounds__(256)
k_pack_w_tiles(const uint4* __restrict__ w_gate, const uint4* __restrict__ w_up, const uint4* __restrict__ w_down,
               uint4* __restrict__ gu, uint4* __restrict__ dt, int n_exp, int H, int I) {
  const int U = I / 64, KB = H / 64, HT = H / 128;
  const size_t per_e = (size_t)I * H / 8;                       // 16-byte pieces per expert and matrix
  const size_t n_gu = 2 * per_e * n_exp, n_d = per_e * n_exp;
  for (size_t o = (size_t)blockIdx.x * blockDim.x + threadIdx.x; o < n_gu + n_d; o += (size_t)gridDim.x * blockDim.x) {
    if (o < n_gu) {
      const int pc = (int)(o & 7), r = (int)((o >> 3) & 127);
      const size_t tile = o >> 10;                              // 1024 pieces per tile
      const int kb = (int)(tile % KB), u = (int)((tile / KB) % U), e = (int)(tile / ((size_t)KB * U));
      const int blk = r >> 5, m = (r >> 4) & 1, i16 = r & 15, lc = pc ^ (r & 7);
      const size_t src = ((size_t)e * I + u * 64 + blk * 16 + i16) * (H / 8) + kb * 8 + lc;
      gu[o] = m ? w_up[src] : w_gate[src];
    } else {
      const size_t q = o - n_gu;
      const int pc = (int)(q & 7), r = (int)((q >> 3) & 127);
      const size_t tile = q >> 10;
      const int kb = (int)(tile % U), ht = (int)((tile / U) % HT), e = (int)(tile / ((size_t)U * HT));
      const int lc = pc ^ (r & 7);
      const size_t src = ((size_t)e * H + ht * 128 + r) * (I / 8) + kb * 8 + lc;
      dt[q] = w_down[src];
    }
  }
}

cudaError_t launch_pack_w_tiles(const void* w_gate, const void* w_up, const void* w_down, void* gu, void* dt, int n_exp,
                                int H, int I, cudaStream_t s) {
  const size_t n = 3 * (size_t)I * H / 8 * n_exp;
  const int grid = (int)((n + 255) / 256 < 148 * 16 ? (n + 255) / 256 : 148 * 16);
  k_pack_w_tiles<<<grid, 256, 0, s>>>(static_cast<const uint4*>(w_gate), static_cast<const uint4*>(w_up),
                                      static_cast<const uint4*>(w_down), static_cast<uint4*>(gu), static_cast<uint4*>(dt),
                                      n_exp, H, I);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------------------
// Token rows of every chunk, gathered into B tiles: [chunk rows padded to 16][H] as [kb][np rows][64 k] swizzled,
// and the chunk's (output row, routing weight) table.  One warp per padded row.
// ---------------------------------------------------------------------------------------------------------
struct GatherArgs {
  const __nv_bfloat16* x;       // [T, H]
  const int32_t* perm;
  const float* topk_w;
  const WorkItem* items;
  const int32_t* n_items;
  __nv_bfloat16* xg;            // gathered tiles
  int32_t* row_of;              // [padded rows] output row of the slot (-1: padding)
  float* w_of;                  // [padded rows] its routing weight
  Dims d;
};

__global__ void __launch_bounds__(256) k_gather_tiles(GatherArgs a) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");            // the selection kernel's tables are complete
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int H = a.d.H, n_items = *a.n_items;
  const int pieces = H / 8;                                      // 16-byte pieces per row
  // four CTAs share a chunk: CTA slice s takes the rows n with (n / 8) % 4 == s, its warp w those with n % 8 == w
  const int slice = blockIdx.x & 3;
  for (int c = blockIdx.x >> 2; c < n_items; c += gridDim.x >> 2) {
    const WorkItem it = a.items[c];
    const int np = pad16(it.n), r0 = chunk_row0(it, c);
    __nv_bfloat16* base = a.xg + (size_t)r0 * H;
    for (int n = slice * 8 + warp; n < np; n += 32) {
      int row = -1;
      float wt = 0.f;
      if (n < it.n) slot_row_weight(a.perm[it.begin + n], a.d.T, a.d.k, a.topk_w, row, wt);
      if (lane == 0) {
        a.row_of[r0 + n] = row;
        a.w_of[r0 + n] = wt;
      }
      const uint4* src = reinterpret_cast<const uint4*>(a.x + (size_t)max(row, 0) * H);
      for (int p = lane; p < pieces; p += 32) {
        const uint4 v = row >= 0 ? __ldg(src + p) : make_uint4(0u, 0u, 0u, 0u);
        const int kb = p >> 3, pc = (p & 7) ^ (n & 7);
        *reinterpret_cast<uint4*>(base + (size_t)kb * np * 64 + n * 64 + pc * 8) = v;
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------------------
// The grouped GEMM
// ---------------------------------------------------------------------------------------------------------
struct TileArgs {
  const __nv_bfloat16* w_tiles;   // [e][tile][kb][16 KB]
  const __nv_bfloat16* b_tiles;   // per chunk: [kb][np rows][64 k], chunk c at row chunk_row0(c) * (n_k * 64) elements
  const WorkItem* items;
  const int32_t* n_items;
  const int32_t* row_of;
  const float* w_of;
  __nv_bfloat16* act;             // kEpiSwiglu: output, per chunk [u][np rows][64 columns] swizzled
  float* y;                       // kEpiCombine: [T, H]
  int32_t* status;
  int n_k;                        // k-blocks of 64: H/64 (A) or I/64 (B)
  int tiles_per_chunk;            // I/64 (A) or H/128 (B)
  int H, I;
};

template <int EPI>
__global__ void __launch_bounds__(kTileThreads, 1) k_grouped_gemm(TileArgs a) {
  extern __shared__ unsigned char tile_smem_raw[];
  // 1024-byte alignment for the swizzled tiles
  unsigned char* smem = tile_smem_raw + ((1024u - (smem_u32(tile_smem_raw) & 1023u)) & 1023u);
  unsigned char* stages = smem;
  int32_t* tab_row = reinterpret_cast<int32_t*>(smem + kTileStages * kStageBytes);      // [4 epilogue warps][128]
  float* tab_w = reinterpret_cast<float*>(tab_row + 4 * kTileChunk);                    // [4][128]
  uint64_t* bars = reinterpret_cast<uint64_t*>(tab_w + 4 * kTileChunk);
  uint64_t* bar_full = bars;                       // [stages] bytes of the stage have landed
  uint64_t* bar_empty = bars + kTileStages;        // [stages] the MMAs reading the stage are done
  uint64_t* bar_dfull = bars + 2 * kTileStages;    // [2] accumulator complete
  uint64_t* bar_dempty = bar_dfull + 2;            // [2] accumulator drained by the epilogue
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_dempty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    for (int i = 0; i < kTileStages; ++i) {
      mbar_init(smem_u32(bar_full + i), 1);
      mbar_init(smem_u32(bar_empty + i), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(bar_dfull + i), 1);
      mbar_init(smem_u32(bar_dempty + i), 4);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"((uint32_t)kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  // Everything above overlaps the preceding kernel; its outputs (work items, token tiles) are complete from here.
  asm volatile("griddepcontrol.wait;" ::: "memory");

  const int TPC = a.tiles_per_chunk, NK = a.n_k;
  const long long n_units = (long long)(*a.n_items) * TPC;
  const int u_lo = (int)(n_units * blockIdx.x / gridDim.x), u_hi = (int)(n_units * (blockIdx.x + 1) / gridDim.x);

  if (warp == 0) {
    // ------------------------------ producer ------------------------------
    const uint64_t pol = stream_policy();
    uint32_t it = 0;
    bool ok = true;
    for (int unit = u_lo; unit < u_hi && ok; ++unit) {
      const int c = unit / TPC, j = unit - c * TPC;
      const WorkItem item = a.items[c];
      const int np = pad16(item.n);
      const __nv_bfloat16* wsrc = a.w_tiles + ((size_t)item.e * TPC + j) * NK * kTileElems;
      const __nv_bfloat16* bsrc = a.b_tiles + (size_t)chunk_row0(item, c) * NK * 64;
      for (int kb = 0; kb < NK; ++kb, ++it) {
        const uint32_t s = it % kTileStages;
        if (!(ok = mbar_wait_warp<32>(smem_u32(bar_empty + s), ((it / kTileStages) & 1) ^ 1, abort_flag, a.status, 31))) break;
        if (lane == 0) {
          const uint32_t full = smem_u32(bar_full + s), dst = smem_u32(stages + (size_t)s * kStageBytes);
          mbar_expect_tx(full, (uint32_t)(kTileBytes + np * 128));
          bulk_g2s_stream(dst, wsrc + (size_t)kb * kTileElems, kTileBytes, full, pol);
          bulk_g2s(dst + kTileBytes, bsrc + (size_t)kb * np * 64, (uint32_t)(np * 128), full);
        }
        __syncwarp();
      }
    }
    if (!ok) {
      // gave up: the copies already issued still land in this CTA's shared memory; give them time before the CTA exits
      for (int i = 0; i < 64; ++i) __nanosleep(1000);
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    uint32_t it = 0, un = 0;
    bool ok = true;
    for (int unit = u_lo; unit < u_hi && ok; ++unit, ++un) {
      const int c = unit / TPC;
      const uint32_t idesc = make_idesc_bf16(pad16(a.items[c].n));
      const uint32_t buf = un & 1;
      if (!(ok = mbar_wait_warp(smem_u32(bar_dempty + buf), ((un >> 1) & 1) ^ 1, abort_flag, a.status, 32))) break;
      tc_fence_after();
      const uint32_t acc = tmem_base + buf * kTileChunk;
      for (int kb = 0; kb < NK; ++kb, ++it) {
        const uint32_t s = it % kTileStages;
        if (!(ok = mbar_wait_warp(smem_u32(bar_full + s), (it / kTileStages) & 1, abort_flag, a.status, 33))) break;
        tc_fence_after();
        const uint32_t base = smem_u32(stages + (size_t)s * kStageBytes);
        const uint64_t da = make_kmajor_sw128_desc(base), db = make_kmajor_sw128_desc(base + kTileBytes);
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4) tc_mma(acc, da + 2 * k4, db + 2 * k4, idesc, (kb | k4) != 0);
        tc_commit(smem_u32(bar_empty + s));
      }
      if (ok) tc_commit(smem_u32(bar_dfull + buf));
    }
  } else {
    // ------------------------------ epilogue ------------------------------
    const int q = warp & 3;                          // this warp's lane quarter of the accumulator
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    uint32_t un = 0;
    int tab_chunk = -1;
    bool ok = true;
    for (int unit = u_lo; unit < u_hi && ok; ++unit, ++un) {
      const int c = unit / TPC, j = unit - c * TPC;
      const WorkItem item = a.items[c];
      const int np = pad16(item.n), r0 = chunk_row0(item, c);
      const uint32_t buf = un & 1;
      if (EPI == kEpiCombine && c != tab_chunk) {
        // (output row, weight) of the chunk's slots: every epilogue warp keeps a copy of its own, refilled at its own pace
        __syncwarp();
        for (int n = lane; n < np; n += 32) {
          tab_row[q * kTileChunk + n] = a.row_of[r0 + n];
          tab_w[q * kTileChunk + n] = a.w_of[r0 + n];
        }
        tab_chunk = c;
        __syncwarp();
      }
      if (!(ok = mbar_wait_warp<32>(smem_u32(bar_dfull + buf), (un >> 1) & 1, abort_flag, a.status, 34))) break;
      tc_fence_after();
      const uint32_t acc = tmem_base + buf * kTileChunk + lane_off;
      if (EPI == kEpiSwiglu) {
        // rows of this warp: [16 gate | 16 up] of intermediate columns j*64 + q*16 + (lane & 15)
        const bool is_gate = lane < 16;
        const int i = q * 16 + (lane & 15);                                   // column inside the tile
        __nv_bfloat16* dst = a.act + (size_t)r0 * a.I + (size_t)j * np * 64;   // this unit's [np][64] tile
        for (int c0 = 0; c0 < np; c0 += 8) {
          float v[8];
          tmem_ld8(acc + c0, v);
#pragma unroll
          for (int t = 0; t < 8; ++t) {
            const float o = __shfl_xor_sync(0xffffffffu, v[t], 16);
            const float g = is_gate ? v[t] : o;
            const float u = is_gate ? o : v[t];
            v[t] = g / (1.f + expf(-g)) * u;
          }
          // lanes 0-15 store slots c0 .. c0+3, lanes 16-31 store c0+4 .. c0+7 (padding slots are zero rows: silu(0) * 0 = 0)
          const int tb = is_gate ? 0 : 4;
#pragma unroll
          for (int t = 0; t < 4; ++t) {
            const int n = c0 + tb + t;
            dst[(size_t)n * 64 + (((i >> 3) ^ (n & 7)) << 3) + (i & 7)] = __float2bfloat16_rn(v[tb + t]);
          }
        }
      } else {
        const int32_t* rows = tab_row + q * kTileChunk;
        const float* wts = tab_w + q * kTileChunk;
        float* ycol = a.y + (size_t)j * 128 + q * 32 + lane;
        for (int c0 = 0; c0 < item.n; c0 += 8) {
          float v[8];
          tmem_ld8(acc + c0, v);
#pragma unroll
          for (int t = 0; t < 8; ++t) {
            const int n = c0 + t;
            if (n < item.n) atomicAdd(ycol + (size_t)rows[n] * a.H, wts[n] * v[t]);
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(bar_dempty + buf));
    }
  }

  // ------------------------------ teardown ------------------------------
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kTmemCols) : "memory");
  }
}

// ---------------------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------------------
bool experts_tile_supported(int hidden, int inter) { return hidden % 128 == 0 && inter % 64 == 0; }
int experts_tile_chunk() { return kTileChunk; }
// Rows of the gathered tables: every slot, plus 16 rows of padding slack per chunk.
size_t experts_tile_rows(size_t slots, size_t max_items) { return slots + 16 * max_items + 16; }

cudaError_t configure_experts_tile() {
  static bool done[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev >= 0 && dev < 64 && done[dev]) return cudaSuccess;
  e = cudaFuncSetAttribute(k_grouped_gemm<kEpiSwiglu>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTileSmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(k_grouped_gemm<kEpiCombine>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTileSmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(k_grouped_gemm<kEpiSwiglu>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(k_grouped_gemm<kEpiCombine>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
  if (e == cudaSuccess && dev >= 0 && dev < 64) done[dev] = true;
  return e;
}

static cudaError_t launch_pdl(const void* fn, dim3 grid, dim3 block, size_t smem, cudaStream_t s, void* arg) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  void* params[1] = {arg};
  return cudaLaunchKernelExC(&cfg, fn, params);
}

// gather, gate/up + SwiGLU, down + combine: three launches chained with programmatic dependent launch
cudaError_t launch_experts_tile(const void* x, const void* gu_tiles, const void* d_tiles, Workspace ws, float* y, Dims d,
                                int grid, cudaStream_t s) {
  GatherArgs g;
  g.x = static_cast<const __nv_bfloat16*>(x);
  g.perm = ws.r.perm;
  g.topk_w = ws.r.topk_w;
  g.items = ws.items;
  g.n_items = ws.n_items;
  g.xg = ws.tile_x;
  g.row_of = ws.tile_row;
  g.w_of = ws.tile_w;
  g.d = d;
  cudaError_t e = launch_pdl(reinterpret_cast<const void*>(&k_gather_tiles), dim3(4 * grid), dim3(256), 0, s, &g);
  if (e != cudaSuccess) return e;
  TileArgs a = {};
  a.items = ws.items;
  a.n_items = ws.n_items;
  a.row_of = ws.tile_row;
  a.w_of = ws.tile_w;
  a.act = ws.tile_act;
  a.y = y;
  a.status = ws.status;
  a.H = d.H;
  a.I = d.I;
  a.w_tiles = static_cast<const __nv_bfloat16*>(gu_tiles);
  a.b_tiles = ws.tile_x;
  a.n_k = d.H / 64;
  a.tiles_per_chunk = d.I / 64;
  e = launch_pdl(reinterpret_cast<const void*>(&k_grouped_gemm<kEpiSwiglu>), dim3(grid), dim3(kTileThreads), kTileSmemBytes, s, &a);
  if (e != cudaSuccess) return e;
  a.w_tiles = static_cast<const __nv_bfloat16*>(d_tiles);
  a.b_tiles = ws.tile_act;
  a.n_k = d.I / 64;
  a.tiles_per_chunk = d.H / 128;
  return launch_pdl(reinterpret_cast<const void*>(&k_grouped_gemm<kEpiCombine>), dim3(grid), dim3(kTileThreads), kTileSmemBytes, s, &a);
}

}  // namespace team
