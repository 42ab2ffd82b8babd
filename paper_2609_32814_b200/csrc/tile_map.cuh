// Tile enumeration of the grouped GEMM, computed inside the GEMM kernels.
//
// Tile classes (ClassRec: pair (i,j), tiles per m-tile, first column, tile width; 8 bytes) are fixed per
// handle and sorted on the host, most expensive first.  Only the number of m-tiles of every row
// type depends on the batch: each CTA turns the bucket offsets (device memory, or arithmetic for
// the cyclic schedule) into the prefix table "tiles before class c" in shared memory and decodes
// tile indices with one binary search and one division.  No tile list is ever written to global
// memory and no extra kernel is needed to produce one.  Inside a class tiles are ordered m-tile
// major, n-tile fastest, so neighbours share their rows.
#pragma once

#include "common.cuh"

namespace algproj {

struct TileMap {
  int n_classes;
  int total;                       // number of tiles
  int q;
  int seq_rounds;                  // tile records precomputed for this worker (the last one is the end marker)
  int seq_valid;                   // tiles this worker owns
  int pad_[1];
  int offsets[kMaxQ + 2];          // bucket offsets (first bucketed row of each type)
  // followed in shared memory by: ClassRec cls[n_classes]; int prefix[n_classes + 1];
  __device__ __forceinline__ ClassRec *cls() { return reinterpret_cast<ClassRec *>(this + 1); }
  __device__ __forceinline__ int *prefix() { return reinterpret_cast<int *>(cls() + n_classes); }
};
static_assert(sizeof(TileMap) % 16 == 0, "class records stay 16-byte aligned behind the header");

__host__ __device__ inline size_t tile_map_bytes(int n_classes) {
  return sizeof(TileMap) + (size_t)n_classes * sizeof(ClassRec) + (size_t)(n_classes + 1) * sizeof(int);
}

// Called by all threads of the CTA (blockDim.x >= 32).  `offsets` = device bucket offsets, or
// nullptr for the cyclic schedule with equal buckets of cyclic_rows rows.  Ends with a barrier.
__device__ inline void tile_map_build(TileMap *tm, const DevTable *tab, const SmallTable &st, int q, int nc,
                                      const int *offsets, int cyclic_rows, int M, const TileGeom &g) {
  if (threadIdx.x == 0) tm->n_classes = nc, tm->q = q;
  for (int t = threadIdx.x; t <= q + 1; t += blockDim.x)
    tm->offsets[t] = offsets ? offsets[t] : (t <= q ? t * cyclic_rows : M);
  __syncthreads();
  ClassRec *cls = tm->cls();
  int *prefix = tm->prefix();
  for (int c = threadIdx.x; c < nc; c += blockDim.x) {
    const ClassRec r = st.valid ? st.cls[c] : tab->cls[c];
    cls[c] = r;
    const int rows = tm->offsets[r.i + 1] - tm->offsets[r.i];
    prefix[c] = ((rows + g.tile_m - 1) >> g.tile_m_log2) * (int)r.n_tiles;
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
  const ClassRec r = tm->cls()[lo];
  const int loc = idx - prefix[lo];
  const int ntl = (int)r.n_tiles, mt = loc / ntl, nt = loc - mt * ntl;
  const int rows = tm->offsets[r.i + 1] - tm->offsets[r.i];
  rec.row0 = tm->offsets[r.i] + (mt << g.tile_m_log2);
  rec.rows = min(g.tile_m, rows - (mt << g.tile_m_log2));
  rec.pair = ((int)r.i * tm->q + (int)r.j) | ((int)r.cols << 16);
  rec.n0 = r.col0 + nt * (int)r.cols;
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
// The tile sequence of one persistent worker is decoded once by the threads of the CTA (one round
// per thread), so that the single-thread roles (TMA producer, MMA issuer) only read a 16-byte
// record per tile.  Rounds beyond `cap` are decoded on the fly.
__device__ __forceinline__ int snake_index(int round, int worker, int n_workers) {
  return round * n_workers + ((round & 1) ? (n_workers - 1 - worker) : worker);
}
// `nkb_of_pair` (optional, shared memory): number of K blocks of the tiles of a pair; it is packed
// into the upper half of TileRec::rows so that the MMA thread needs nothing but the record.
__device__ __forceinline__ TileRec tile_seq_decode(TileMap *tm, const TileGeom &g, int pos, int worker, int n_workers,
                                                   const uint16_t *nkb_of_pair) {
  const int n = tm->seq_valid;
  TileRec rec;
  if (pos >= n) {
    rec.row0 = -1, rec.rows = 0, rec.pair = 0, rec.n0 = 0;
    return rec;
  }
  rec = tile_map_decode(tm, g, snake_index(pos, worker, n_workers));
  if (nkb_of_pair && rec.row0 >= 0) rec.rows |= (int)nkb_of_pair[rec.pair & 0xFFFF] << 16;
  return rec;
}
__device__ inline void tile_seq_build(TileRec *recs, int cap, TileMap *tm, const TileGeom &g, int worker, int n_workers,
                                      const uint16_t *nkb_of_pair = nullptr) {
  // rounds this worker can have at all: ceil(total / n_workers), plus one record that marks the end
  const int all_rounds = (tm->total + n_workers - 1) / n_workers;
  const int valid = all_rounds == 0 ? 0 : all_rounds - 1 + (snake_index(all_rounds - 1, worker, n_workers) < tm->total);
  const int rounds = min(cap, valid + 1);
  if (threadIdx.x == 0) tm->seq_rounds = rounds, tm->seq_valid = valid;
  __syncthreads();
  for (int r = threadIdx.x; r < rounds; r += blockDim.x) recs[r] = tile_seq_decode(tm, g, r, worker, n_workers, nkb_of_pair);
  __syncthreads();
}
__device__ __forceinline__ TileRec tile_seq_get(const TileRec *recs, TileMap *tm, const TileGeom &g, int round, int worker,
                                                int n_workers, const uint16_t *nkb_of_pair = nullptr) {
  if (round < tm->seq_rounds) return recs[round];
  return tile_seq_decode(tm, g, round, worker, n_workers, nkb_of_pair);
}

// The whole plan of one worker -- class prefix table and its own tile sequence, K-block counts
// included -- built by ONE warp with warp-level synchronisation only, so that the other warps of
// the CTA can set up barriers and tensor memory meanwhile and a single CTA barrier ends the
// prologue.  `keep` / `so` are read from the by-value table when it is valid, else from `tab`.
// `seg_rows` (optional): every reduction segment has this many rows (weight-gradient pass, cyclic schedule).
// `dyn_so` (optional, device memory): offsets of the reduction segments when they are not the
// table's (weight-gradient pass: padded row buckets).
__device__ inline void tile_plan_warp(TileMap *tm, TileRec *recs, int cap, const DevTable *tab, const SmallTable &st,
                                      int q, int nc, const int *offsets, int cyclic_rows, int M, const TileGeom &g,
                                      int worker, int n_workers, int k_block, const int *dyn_so = nullptr, int seg_rows = 0) {
  const int lane = threadIdx.x & 31;
  if (lane == 0) tm->n_classes = nc, tm->q = q;
  for (int t = lane; t <= q + 1; t += 32) tm->offsets[t] = offsets ? offsets[t] : (t <= q ? t * cyclic_rows : M);
  __syncwarp();
  ClassRec *cls = tm->cls();
  int *prefix = tm->prefix();
  int carry = 0;
  for (int c0 = 0; c0 < nc; c0 += 32) {
    const int c = c0 + lane;
    int v = 0;
    if (c < nc) {
      const ClassRec r = st.valid ? st.cls[c] : tab->cls[c];
      cls[c] = r;
      const int rows = tm->offsets[r.i + 1] - tm->offsets[r.i];
      v = ((rows + g.tile_m - 1) >> g.tile_m_log2) * (int)r.n_tiles;
    }
    int incl = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += n;
    }
    if (c < nc) prefix[c] = carry + incl - v;
    carry += __shfl_sync(0xffffffffu, incl, 31);
  }
  const int total = carry;
  const int all_rounds = (total + n_workers - 1) / n_workers;
  const int valid = all_rounds == 0 ? 0 : all_rounds - 1 + (snake_index(all_rounds - 1, worker, n_workers) < total);
  const int rounds = min(cap, valid + 1);
  if (lane == 0) prefix[nc] = total, tm->total = total, tm->seq_rounds = rounds, tm->seq_valid = valid;
  __syncwarp();
  for (int r = lane; r < rounds; r += 32) {
    TileRec rec = tile_seq_decode(tm, g, r, worker, n_workers, nullptr);
    if (rec.row0 >= 0) {
      const int pr = rec.pair & 0xFFFF;
      const uint32_t mask = st.valid ? st.keep[pr] : tab->keep[pr];
      int n = 0;
      for (int k = 0; k < q; ++k)
        if ((mask >> k) & 1u)
          n += (seg_rows ? seg_rows : dyn_so ? dyn_so[k + 1] - dyn_so[k] : st.valid ? st.so[k + 1] - st.so[k] : tab->so[k + 1] - tab->so[k]) / k_block;
      rec.rows |= n << 16;
    }
    recs[r] = rec;
  }
}

}  // namespace algproj
