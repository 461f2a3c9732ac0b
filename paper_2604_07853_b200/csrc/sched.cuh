// Static persistent tile schedule over ragged row groups (one group of rows per expert), kept in
// shared memory: off[e] = first row of expert e, prefix[e] = tiles before expert e.
#pragma once
#include <stdint.h>

namespace qarl {

struct TileCoord {
  int e, n_tile, m0, m_end;
};

// Tile T -> (expert, column tile, first row, end of the expert's rows).  Within an expert the
// row tiles vary fastest, so CTAs running at the same time share one weight tile through L2.
// cur_e only moves forward: a caller walks its tiles in ascending order.
__device__ __forceinline__ TileCoord decode_tile(const int32_t* off, const int32_t* prefix, int rows_per_tile, int T,
                                                 int& cur_e) {
  while (T >= prefix[cur_e + 1]) ++cur_e;
  const int local = T - prefix[cur_e];
  const int rows = off[cur_e + 1] - off[cur_e];
  const int m_tiles = (rows + rows_per_tile - 1) / rows_per_tile;
  TileCoord c;
  c.e = cur_e;
  c.n_tile = local / m_tiles;
  c.m0 = off[cur_e] + (local % m_tiles) * rows_per_tile;
  c.m_end = off[cur_e + 1];
  return c;
}

// Fills off[0..E] from the device offsets (or one dense group) and prefix[0..E] with the
// exclusive scan of tiles per expert.  Called by every thread of the CTA; contains barriers.
// Boundaries are forced into [0, rows_total] and a group that ends before it starts gets no
// tile, so whatever the offsets array holds, no tile reaches outside the tensors.
__device__ __forceinline__ void build_tile_list(int32_t* off, int32_t* prefix, const int32_t* offsets, int rows_total,
                                                int E, int rows_per_tile, int n_tiles) {
  for (int e = threadIdx.x; e <= E; e += blockDim.x)
    off[e] = offsets ? min(max(offsets[e], 0), rows_total) : (e == 0 ? 0 : rows_total);
  __syncthreads();
  if (threadIdx.x < 32) {
    const int lane = threadIdx.x;
    int carry = 0;
    for (int base = 0; base < E; base += 32) {
      const int e = base + lane;
      int v = 0;
      if (e < E) v = ((max(off[e + 1] - off[e], 0) + rows_per_tile - 1) / rows_per_tile) * n_tiles;
      int inc = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int u = __shfl_up_sync(0xFFFFFFFFu, inc, o);
        if (lane >= o) inc += u;
      }
      if (e < E) prefix[e] = carry + inc - v;
      carry += __shfl_sync(0xFFFFFFFFu, inc, 31);
    }
    if (lane == 0) prefix[E] = carry;
  }
  __syncthreads();
}

// With W = ceil(tiles / CTAs) rounds, ceil(tiles / W) CTAs already finish in W rounds; using
// exactly that many keeps every round full.  The CTAs beyond that count retire at once.
__device__ __forceinline__ int balanced_cta_count(int total_tiles, int grid) {
  if (total_tiles <= 0) return grid;
  const int rounds = (total_tiles + grid - 1) / grid;
  return (total_tiles + rounds - 1) / rounds;
}

}  // namespace qarl
