// Tile enumeration of the grouped GEMM, computed inside the GEMM kernels.
//
// Every CTA builds, once at start-up and in shared memory, the prefix table "tiles before tile
// class c" from the bucket offsets (row counts per type, which only exist on the device) and the
// handle's class order (most expensive class first), and then decodes tile indices on the fly.
// No tile list is ever written to global memory and no extra kernel is needed to produce one.
//
// A tile class is (pair (i,j), w): w = 0 -> tiles of the full tile width inside output group j,
// w = 1 -> the narrower remainder tile of that group (only when the kernel splits remainders).
// Inside a class tiles are ordered m-tile major, n-tile fastest, so neighbours share their rows.
#pragma once

#include "common.cuh"

namespace algproj {

struct TileMap {
  int n_classes;
  int total;                       // number of tiles
  int q;
  int offsets[kMaxQ + 2];          // bucket offsets (first bucketed row of each type)
  int ro[kMaxQ + 1];               // output group offsets
  // followed in shared memory by: int cls[n_classes]; int prefix[n_classes + 1];
  __device__ __forceinline__ int *cls() { return reinterpret_cast<int *>(this + 1); }
  __device__ __forceinline__ int *prefix() { return cls() + n_classes; }
};

__host__ __device__ inline size_t tile_map_bytes(int n_classes) {
  return sizeof(TileMap) + (size_t)(2 * n_classes + 1) * sizeof(int);
}

__device__ __forceinline__ int tile_map_n_tiles(const TileGeom &g, int cls, int width) {
  const int w = cls & 1;
  if (!g.split_rem) return w == 0 ? ceil_div(width, g.tile_n) : 0;
  return w == 0 ? width / g.tile_n : ((width % g.tile_n) ? 1 : 0);
}

// Called by all threads of the CTA (blockDim.x >= 32).  `offsets` = device bucket offsets, or
// nullptr for the cyclic schedule with equal buckets of cyclic_rows rows.  Ends with a barrier.
__device__ inline void tile_map_build(TileMap *tm, const DevTable *tab, const SmallTable &st, int q, int nc,
                                      const int *offsets, int cyclic_rows, int M, const TileGeom &g) {
  if (threadIdx.x == 0) tm->n_classes = nc, tm->q = q;
  for (int t = threadIdx.x; t <= q + 1; t += blockDim.x)
    tm->offsets[t] = offsets ? offsets[t] : (t <= q ? t * cyclic_rows : M);
  for (int t = threadIdx.x; t <= q; t += blockDim.x) tm->ro[t] = st.valid ? st.ro[t] : tab->ro[t];
  __syncthreads();
  int *cls = tm->cls(), *prefix = tm->prefix();
  for (int c = threadIdx.x; c < nc; c += blockDim.x) {
    const int id = st.valid ? st.class_order[c] : tab->class_order[c];
    const int pair = id >> 1, i = pair / q, j = pair % q;
    cls[c] = id;
    prefix[c] = ceil_div(tm->offsets[i + 1] - tm->offsets[i], g.tile_m) * tile_map_n_tiles(g, id, tm->ro[j + 1] - tm->ro[j]);
  }
  __syncthreads();
  if (threadIdx.x < 32) {  // exclusive scan of the counts by one warp
    const int lane = threadIdx.x;
    int carry = 0;
    for (int c0 = 0; c0 < nc; c0 += 32) {
      const int c = c0 + lane;
      const int v = c < nc ? prefix[c] : 0;
      int incl = v;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += n;
      }
      if (c < nc) prefix[c] = carry + incl - v;
      carry += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) prefix[nc] = carry, tm->total = carry;
  }
  __syncthreads();
}

// Tile `idx` (0 <= idx < total): rows [row0, row0+rows) of the bucketed order, columns
// [n0, n0 + cols) with cols packed into pair's upper half.  idx >= total gives row0 = -1.
__device__ __forceinline__ TileRec tile_map_decode(TileMap *tm, const TileGeom &g, int idx) {
  TileRec rec;
  if (idx >= tm->total) {
    rec.row0 = -1, rec.rows = 0, rec.pair = 0, rec.n0 = 0;
    return rec;
  }
  const int *prefix = tm->prefix();
  int lo = 0, hi = tm->n_classes;  // prefix[lo] <= idx < prefix[hi]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (prefix[mid] <= idx) lo = mid; else hi = mid;
  }
  const int id = tm->cls()[lo];
  const int q = tm->q, pair = id >> 1, i = pair / q, j = pair % q;
  const int width = tm->ro[j + 1] - tm->ro[j];
  const int n_tiles = tile_map_n_tiles(g, id, width);
  const int loc = idx - prefix[lo];
  const int mt = loc / n_tiles, nt = loc % n_tiles;
  const int rows = tm->offsets[i + 1] - tm->offsets[i];
  const int c0 = (g.split_rem && (id & 1)) ? (width / g.tile_n) * g.tile_n : nt * g.tile_n;
  rec.row0 = tm->offsets[i] + mt * g.tile_m;
  rec.rows = min(g.tile_m, rows - mt * g.tile_m);
  rec.pair = pair | (min(g.tile_n, width - c0) << 16);
  rec.n0 = tm->ro[j] + c0;
  return rec;
}

// Static schedule: the tile enumeration is sorted most-expensive first; worker c of n takes, in
// round r, tile r*n + c on even rounds and r*n + (n-1-c) on odd rounds (boustrophedon).  That
// balances the per-worker cost like a longest-processing-time assignment without inter-CTA
// traffic, and keeps the workers of one round on neighbouring tiles (same rows or same columns),
// so the lines one CTA pulls into L2 are the lines its neighbours ask for at the same moment.
// (Giving each worker a contiguous run of tiles instead was measured 10-15 % slower: the
// concurrent working set then spreads over the whole problem.)
//
// The tile sequence of one persistent worker, decoded once by all threads of the CTA so that the
// single-thread roles (TMA producer, MMA issuer) only read a 16-byte record per tile: their
// instruction streams share a scheduler with busy epilogue warps, which makes scalar work in them
// several times more expensive than it looks.  Rounds beyond `cap` are decoded on the fly.
__device__ __forceinline__ int snake_index(int round, int worker, int n_workers) {
  return round * n_workers + ((round & 1) ? (n_workers - 1 - worker) : worker);
}
__device__ inline void tile_seq_build(TileRec *recs, int cap, TileMap *tm, const TileGeom &g, int worker,
                                      int n_workers) {
  for (int r = threadIdx.x; r < cap; r += blockDim.x) recs[r] = tile_map_decode(tm, g, snake_index(r, worker, n_workers));
  __syncthreads();
}
__device__ __forceinline__ TileRec tile_seq_get(const TileRec *recs, int cap, TileMap *tm, const TileGeom &g, int round,
                                                int worker, int n_workers) {
  if (round < cap) return recs[round];
  return tile_map_decode(tm, g, snake_index(round, worker, n_workers));
}

}  // namespace algproj
