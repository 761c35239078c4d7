// team_pack_w_down: one-time conversion of the down-projection weights into the layout the expert
// kernels read.
//
// Eq. 1's expert FFN multiplies W_down [H, I] with the activation vector of length I.  The expert
// kernels cut I into groups of 16 columns and give every group to exactly one CTA, so a CTA needs,
// for each of its groups, the 16 columns of all H rows.  In the row-major matrix those are H pieces
// of 32 bytes (bf16) at a stride of 2*I bytes; stored group by group ([I/16][H][16]) they are one
// contiguous block of 32*H bytes that streams from HBM at full rate.
#include "team_common.cuh"

namespace team {

// One thread per 16-byte piece: consecutive threads read consecutive pieces of a source row.
__global__ void __launch_bounds__(256) k_pack_w_down(const uint4* __restrict__ src, uint4* __restrict__ dst, long long n_pieces,
                                                      int H, int pieces_per_row, int pieces_per_group) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= n_pieces) return;
  const long long row = idx / pieces_per_row;            // e * H + h
  const int p = (int)(idx - row * pieces_per_row);
  const long long e = row / H;
  const int h = (int)(row - e * H);
  const int grp = p / pieces_per_group, r = p - grp * pieces_per_group;
  const int groups = pieces_per_row / pieces_per_group;
  dst[((e * groups + grp) * H + h) * pieces_per_group + r] = src[idx];
}

}  // namespace team

extern "C" int team_pack_w_down(const void* src, void* dst, int n_experts_total, int hidden, int inter, int dtype,
                                void* stream) {
  if (src == nullptr || dst == nullptr || src == dst) return TEAM_ERR_ARG;
  if (((uintptr_t)src & 15) || ((uintptr_t)dst & 15)) return TEAM_ERR_ARG;
  if (n_experts_total <= 0 || hidden <= 0 || inter <= 0 || inter % 16) return TEAM_ERR_SHAPE;
  if (dtype != TEAM_DTYPE_F32 && dtype != TEAM_DTYPE_BF16) return TEAM_ERR_SHAPE;
  const int elt = dtype == TEAM_DTYPE_F32 ? 4 : 2;
  const int pieces_per_row = inter * elt / 16, pieces_per_group = 16 * elt / 16;
  const long long n_pieces = (long long)n_experts_total * hidden * pieces_per_row;
  const long long blocks = (n_pieces + 255) / 256;
  if (blocks > 0x7fffffffLL) return TEAM_ERR_SHAPE;
  team::k_pack_w_down<<<(unsigned)blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const uint4*>(src), static_cast<uint4*>(dst), n_pieces, hidden, pieces_per_row, pieces_per_group);
  return cudaGetLastError() == cudaSuccess ? TEAM_OK : TEAM_ERR_CUDA;
}

extern "C" int team_pack_w_tiles(const void* w_gate, const void* w_up, const void* w_down, void* gu_tiles, void* down_tiles,
                                 int n_experts_total, int hidden, int inter, void* stream) {
  if (!w_gate || !w_up || !w_down || !gu_tiles || !down_tiles) return TEAM_ERR_ARG;
  if (gu_tiles == w_gate || gu_tiles == w_up || down_tiles == w_down || gu_tiles == down_tiles) return TEAM_ERR_ARG;
  if (((uintptr_t)w_gate & 15) || ((uintptr_t)w_up & 15) || ((uintptr_t)w_down & 15) || ((uintptr_t)gu_tiles & 127) ||
      ((uintptr_t)down_tiles & 127))
    return TEAM_ERR_ARG;
  if (n_experts_total <= 0 || hidden <= 0 || inter <= 0 || hidden % 128 || inter % 64) return TEAM_ERR_SHAPE;
  const cudaError_t e = team::launch_pack_w_tiles(w_gate, w_up, w_down, gu_tiles, down_tiles, n_experts_total, hidden, inter,
                                                  static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? TEAM_OK : TEAM_ERR_CUDA;
}
