// Large-algebra grouped GEMM for sm_100a: the complete-graph law Q_q with q equal groups, q up to
// 256, and group widths that need not be multiples of the GPU tile (the fixed-block regime of
// Section "Kernel Benchmarks" and the appendix "Large Projections and Square Products": blocks such
// as 160 x 800, 80 x 400, 40 x 200, or b x b blocks with q = n / b).
//
// One output tile = up to 128 rows of one row type i  x  tile_n columns of one output group j.  Its
// reduction is x_i W_ij + x_j W_jj (Eqs. typed-diag / typed-off; one product when i = j), both
// summed in the same TMEM accumulator -- the paper's two stages (diagonal maps for all rows, then
// the type-dependent maps) become two reduction segments of one tile, so Y is written exactly once
// and never read.
//
// What differs from the table-driven kernel (proj_tc.cu):
//  * No interaction table and no tile classes: with 65536 (type, group) pairs neither fits shared
//    memory.  Tile t is decoded by arithmetic, type-major: all tiles of type i are consecutive, so
//    the row panel W[S_i, :] -- which only type-i rows use -- streams from HBM once while the
//    q diagonal blocks stay in L2; inside a type the m-tile index runs fastest (CTAs working side by
//    side share their B blocks), then the column tile, then the output group.
//  * Operands come through PER-GROUP tensor maps: X as {s, q, rows} (or {s, q, q, M/q} for the
//    cyclic schedule), W as {N, s, q}.  Coordinates past a group's width (or past N) read as
//    zero, so a group that is narrower than the pipeline stage, and a last column tile narrower
//    than tile_n, are padded for free: extra multiply-adds on zeros, no extra bytes, no repacked
//    copies of X or W.  Everything stays 16-byte aligned because widths are multiples of 8.
//  * The MMA width is a launch parameter (tile_n, a multiple of 16), stores are masked per 8
//    columns.
//  * Group widths that are multiples of 4 but not of 8 (20 x 100: the q = 256 split of 5120 -> 25600) cannot be
//    addressed by tensor maps (boxes start on 16 bytes).  For those the caller of this file repacks X and W with
//    every group widened to the next multiple of 8 (zeros; pad_groups_kernel in bucket.cu) and passes the
//    repacked widths as s, r and the width of Y's groups as r_out; stores then go in 8-byte pieces.  (Staging the
//    unpadded operands with 8-byte asynchronous copies from two producer warps was built first: bit-exact, but
//    each copy instruction took ~200 cycles to issue with the loads missing L2, 2-10 x slower than repacking.)
//  * Types with at most 64 rows (large q at moderate M) would leave most of a 128-row tile empty, and every
//    tile costs its epilogue and its hand-overs whatever it holds.  With equal buckets a tile then takes
//    P = 128 / rows-per-type consecutive types: ONE diagonal segment x_j W_jj for all its rows (the map is the
//    same for every type), then one panel segment x_i W_ij per type i != j whose A block is fetched through a
//    view {s, group, row in type, type} with a 128-row box placed so that type i's rows land where they sit in
//    the tile and every other row is out of range, i.e. zero: the product adds nothing to the other types'
//    rows.  1 + P segments and one epilogue instead of 2 P segments and P epilogues.
//  * Output groups of at most 128 columns (25600 -> 5120 in 64 ... 256 groups) make narrow tiles that cost their
//    hand-overs and their A fetches like wide ones.  A tile then covers G = floor(256 / r) consecutive groups: the
//    panel product x_i W[S_i, all its columns] is ONE segment, and each group g adds its diagonal product
//    x_j W_jj as a full-width product whose B block is zero outside the group's columns -- fetched through a view of
//    the bank by {column in group, column group, k, row group} with the box started at a negative column, so the
//    out-of-range columns are the zeros.  1 + G segments for G groups instead of 2 G, and G times fewer tiles.
//  * What bounds operand fill on one SM is the number of row requests the copy engine makes (about one
//    row of up to 128 bytes every two cycles), not their bytes.  So a stage is always fetched in rows of
//    128 bytes (64-deep stages, even for groups narrower than 64: the rest of the row is zero fill), only
//    the 64-column boxes of W the tile width needs are requested, and when no row type has 128 rows the box
//    of X is cut to the rows there are (the MMA still spans 128 rows; the unused ones are never stored).
// Warp roles as in proj_tc.cu: warp 0 = TMA producer of A, warp 10 = TMA producer of B, warp 1 =
// TMEM allocator + MMA issuer, warps 2..9 = epilogue (TMEM lane quadrant = warp % 4; the two warps
// of a quadrant alternate over the 32-column chunks).  Double-buffered accumulator; every wait is
// bounded and ends in ALG_ERR_DEVICE_TIMEOUT.
#include <cudaTypedefs.h>

#include <algorithm>

#include "tc_common.cuh"

namespace algproj {

using namespace tc;

ALG_TRACE_DEFINE(proj_big)

namespace {

constexpr int kThreads = 352;
constexpr int kEpiWarps = 8;
constexpr int kProducerWarpB = 10;
constexpr int kStoreBufBytes = 32 * 64;   // per epilogue warp: 32 rows x 32 bf16 columns

struct Ctl {
  uint64_t full[12];
  uint64_t empty[12];
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint32_t tmem_base;
  volatile int abort_flag;
  long long wait_limit;
  int total;                    // tiles of the launch
  int off[kBigMaxQ + 1];        // sched 0: first bucketed row of every type
  int pre[kBigMaxQ + 1];        // sched 0: tiles before type i
};

__device__ __noinline__ bool wait_slow(uint32_t bar, uint32_t parity, Ctl *ctl, int *status) {
  const long long t0 = clock64();
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 255u) == 0) {
      if (ctl->abort_flag) return false;
      if (clock64() - t0 > ctl->wait_limit) {
        ctl->abort_flag = 1;
        atomicExch(status, (int)ALG_ERR_DEVICE_TIMEOUT);
        return false;
      }
    }
  }
  return true;
}
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, Ctl *ctl, int *status) {
  if (mbar_try_wait(bar, parity)) return true;
  return wait_slow(bar, parity, ctl, status);
}

template <int TILE_N, int BK>
struct Cfg {
  static constexpr int kABytes = 128 * BK * 2;
  static constexpr int kBChunkBytes = BK * 64 * 2;              // one BK(k) x 64(n) box
  static constexpr int kChunks = TILE_N / 64;
  static constexpr int kStageBytes = kABytes + kBChunkBytes * kChunks;
  static constexpr int kStages = (192 * 1024) / kStageBytes > 12 ? 12 : (192 * 1024) / kStageBytes;
  static constexpr int kTmemCols = 2 * TILE_N;
  static constexpr uint32_t kSwzK = BK == 64 ? 2 : 4;
  static constexpr uint32_t kSboK = 8 * BK * 2;
  static constexpr int kSmemBytes = kStages * kStageBytes + kEpiWarps * kStoreBufBytes + (int)sizeof(Ctl) + 1024;
  static_assert(BK == 64 || BK == 32, "stage depth");
  static_assert(TILE_N == 128 || TILE_N == 256, "stage width");
};

struct Tile {
  int row0, rows;   // bucketed rows [row0, row0 + rows), all of type i; row0 < 0: no more tiles
  int i, j;         // packed tiles: i = first of np consecutive types; j = first of ng consecutive output groups
  int np, ng;
  int n0, cols;     // absolute first column in Y, valid columns (<= tile_n)
  int n0_w;         // first column in the bank (differs from n0 when the bank's groups are padded)
};

// t / d for 0 <= t < 2^22 with the reciprocal of d from the host: the tile decode runs once per tile in every role, and
// tiles of this path are short -- an integer division is a few dozen dependent instructions
__device__ __forceinline__ int fast_div(int t, int d, float inv_d) {
  if (inv_d == 0.f) return t / d;
  int qt = (int)(((float)t + 0.5f) * inv_d);
  if (qt * d > t) --qt;
  if ((qt + 1) * d <= t) ++qt;
  return qt;
}

// Tile t of the launch (uniform across the warp).  Type-major; inside a type: m-tile fastest, then
// the column tile, then the output group.
__device__ __forceinline__ Tile decode_tile(const BigArgs &a, const Ctl *ctl, int t) {
  Tile o;
  o.row0 = -1, o.rows = 0, o.i = 0, o.j = 0, o.n0 = 0, o.cols = 0, o.n0_w = 0, o.np = 1, o.ng = 1;
  if (t >= ctl->total) return o;
  if (a.pack > 1 && a.gpack > 1) {
    // several types AND several output groups per tile.  Type-group major; inside a type group first the column
    // units (a.gpack groups each) that hold none of its types, one tile each, then the groups of the other units
    // one by one (a tile never holds a type together with other groups than its own: the diagonal product of
    // group k and the panel product of type k would both carry x_k W_kk)
    int lo = 0, hi = a.n_tg;   // pre[lo] <= t < pre[hi]
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (ctl->pre[mid] <= t) lo = mid; else hi = mid;
    }
    const int l = t - ctl->pre[lo], g = a.gpack;
    o.i = lo * a.pack;
    o.np = min(a.pack, a.q - o.i);
    const int n_units = a.n_units, ua = fast_div(o.i, g, a.inv_g), ub = fast_div(o.i + o.np - 1, g, a.inv_g), apart = n_units - (ub - ua + 1);
    if (l < apart) {
      o.j = (l < ua ? l : l + (ub - ua + 1)) * g;
      o.ng = min(g, a.q - o.j);
    } else {
      o.j = ua * g + (l - apart);
      o.ng = 1;
    }
    o.row0 = o.i * a.rows_per_type;
    o.rows = o.np * a.rows_per_type;
    o.n0 = o.j * a.r_out;
    o.n0_w = o.j * a.r;
    o.cols = o.ng * a.r;
    return o;
  }
  if (a.pack > 1) {   // type-group major, then the output group, then the column tile
    const int per_group = a.q * a.nt_n;
    const int tg = fast_div(t, per_group, a.inv_per_type), rem = t - tg * per_group;
    const int j = a.nt_n == 1 ? rem : rem / a.nt_n, nt = rem - j * a.nt_n;
    o.i = tg * a.pack, o.j = j;
    o.np = min(a.pack, a.q - o.i);
    o.row0 = o.i * a.rows_per_type;
    o.rows = o.np * a.rows_per_type;
    o.n0 = j * a.r_out + nt * a.tile_n;
    o.n0_w = j * a.r + nt * a.tile_n;
    o.cols = min(a.tile_n, a.r_out - nt * a.tile_n);
    return o;
  }
  int i, rem, base, rows_i;
  if (a.sched != 0) {
    rows_i = a.rows_per_type;
    const int per_type = ((rows_i + 127) >> 7) * a.col_units;
    i = fast_div(t, per_type, a.inv_per_type);
    rem = t - i * per_type;
    base = i * rows_i;
  } else {
    int lo = 0, hi = a.q;   // pre[lo] <= t < pre[hi]
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (ctl->pre[mid] <= t) lo = mid; else hi = mid;
    }
    i = lo;
    rem = t - ctl->pre[i];
    base = ctl->off[i];
    rows_i = ctl->off[i + 1] - base;
  }
  const int mt_i = (rows_i + 127) >> 7;
  const int u = mt_i == 1 ? rem : rem / mt_i, mt = rem - u * mt_i;
  o.row0 = base + (mt << 7);
  o.rows = min(128, rows_i - (mt << 7));
  if (a.gpack > 1) {   // a tile of several whole output groups
    o.i = i, o.j = u * a.gpack;
    o.ng = min(a.gpack, a.q - o.j);
    o.n0 = o.j * a.r_out;
    o.n0_w = o.j * a.r;
    o.cols = o.ng * a.r;   // columns of the accumulator in use (groups at their width in the bank)
    return o;
  }
  const int j = a.nt_n == 1 ? u : u / a.nt_n, nt = u - j * a.nt_n;
  o.i = i, o.j = j;
  o.n0 = j * a.r_out + nt * a.tile_n;
  o.n0_w = j * a.r + nt * a.tile_n;
  o.cols = min(a.tile_n, a.r_out - nt * a.tile_n);
  return o;
}

template <int TILE_N, int BK>
__global__ void __launch_bounds__(kThreads, 1)
proj_big_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmA2,
                const __grid_constant__ CUtensorMap tmB, const __grid_constant__ CUtensorMap tmB2, const BigArgs a) {
  using C = Cfg<TILE_N, BK>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t *store_buf = smem + C::kStages * C::kStageBytes;
  Ctl *ctl = (Ctl *)(store_buf + kEpiWarps * kStoreBufBytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q = a.q;
  ALG_TRACE_VARS;
  ALG_TRACE_CTA(0, 0);
  if (threadIdx.x == 0) ALG_TRACE(0, 20);

  if (warp == 0) {
    if (lane < C::kStages) {
      mbar_init(smem_u32(&ctl->full[lane]), 1);
      mbar_init(smem_u32(&ctl->empty[lane]), 1);
    } else if (lane < C::kStages + 2) {
      mbar_init(smem_u32(&ctl->tmem_full[lane - C::kStages]), 1);
      mbar_init(smem_u32(&ctl->tmem_empty[lane - C::kStages]), kEpiWarps);
    } else if (lane == 31) {
      ctl->abort_flag = 0;
      ctl->wait_limit = a.wait_limit;
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  } else if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)),
                 "r"((uint32_t)C::kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  } else if (warp == 3 && lane == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmA) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmB) : "memory");
    if (a.pack > 1) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmA2) : "memory");
    if (a.gpack > 1) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmB2) : "memory");
  }
  // Everything above touches only this CTA's own state and may overlap the previous kernel of the stream.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (warp == 2) {
    // tile counts: one warp turns the bucket offsets into "tiles before type i"
    if (a.pack > 1 && a.gpack > 1) {
      // tiles before every type group (see decode_tile)
      const int n_tg = (q + a.pack - 1) / a.pack, g = a.gpack, n_units = (q + g - 1) / g;
      int carry = 0;
      for (int t0 = 0; t0 < n_tg; t0 += 32) {
        const int tg = t0 + lane;
        int v = 0;
        if (tg < n_tg) {
          const int i0 = tg * a.pack, np = min(a.pack, q - i0), ua = i0 / g, ub = (i0 + np - 1) / g;
          v = n_units - (ub - ua + 1) + (min(q, (ub + 1) * g) - ua * g);
        }
        int incl = v;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
          const int n = __shfl_up_sync(0xffffffffu, incl, d);
          if (lane >= d) incl += n;
        }
        if (tg < n_tg) ctl->pre[tg] = carry + incl - v;
        carry += __shfl_sync(0xffffffffu, incl, 31);
      }
      if (lane == 0) ctl->pre[n_tg] = carry, ctl->total = carry;
    } else if (a.pack > 1) {
      if (lane == 0) ctl->total = ((q + a.pack - 1) / a.pack) * q * a.nt_n;
    } else if (a.sched != 0) {
      if (lane == 0) ctl->total = q * ((a.rows_per_type + 127) >> 7) * a.col_units;
    } else {
      int carry = 0;
      for (int i0 = 0; i0 < q; i0 += 32) {
        const int i = i0 + lane;
        int v = 0;
        if (i < q) {
          const int lo = a.offsets[i], hi = a.offsets[i + 1];
          ctl->off[i] = lo;
          if (i == q - 1) ctl->off[q] = hi;
          v = ((hi - lo + 127) >> 7) * a.col_units;
        }
        int incl = v;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
          const int n = __shfl_up_sync(0xffffffffu, incl, d);
          if (lane >= d) incl += n;
        }
        if (i < q) ctl->pre[i] = carry + incl - v;
        carry += __shfl_sync(0xffffffffu, incl, 31);
      }
      if (lane == 0) ctl->pre[q] = carry, ctl->total = carry;
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;
  if (threadIdx.x == 0) ALG_TRACE(0, 24);
  const int nkb_seg = (a.s + BK - 1) / BK;   // pipeline stages per reduction segment (the last one zero-padded)

  if (warp == 0 || warp == kProducerWarpB) {
    // ---------------- TMA producers (warp-uniform loops, one elected lane issues) ----------------
    const bool loads_a = warp == 0;
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    const uint32_t full0 = smem_u32(&ctl->full[0]), empty0 = smem_u32(&ctl->empty[0]);
    const uint32_t smem0 = smem_u32(smem);
    const int b_chunks = a.gated_f ? 2 * a.n_chunks : a.n_chunks;   // 64-column boxes of the bank per stage
    const uint32_t stage_tx = (uint32_t)(a.a_box_rows * BK * 2 + b_chunks * C::kBChunkBytes);   // bytes the copies of a stage deliver
    for (int t = blockIdx.x; ok; t += gridDim.x) {
      const Tile tl = decode_tile(a, ctl, t);
      if (tl.row0 < 0) break;
      if (loads_a && lane == 0) ALG_TRACE(0, 1);
      const bool packed = a.pack > 1;
      // packed tile: segment 0 is the diagonal one (group j), then one panel segment per type of the tile other than j
      const int j_in = packed && tl.ng == 1 && tl.j >= tl.i && tl.j < tl.i + tl.np ? 1 : 0;
      // tile of several output groups: segment 0 is the panel product (k = i), then one diagonal product per group other than i
      const bool gp = a.gpack > 1;
      // several types and several groups: one panel segment per type, then one diagonal segment per group (all rows)
      const bool pg = packed && gp;
      const int i_in = gp && !packed && tl.i >= tl.j && tl.i < tl.j + tl.ng ? 1 : 0;
      const int n_seg = pg ? tl.ng + tl.np - j_in : packed ? 1 + tl.np - j_in : gp ? 1 + tl.ng - i_in : (tl.i == tl.j ? 1 : 2);
      const int a_row = a.sched == 2 ? tl.row0 - tl.i * a.rows_per_type : tl.row0;
      for (int sg = 0; sg < n_seg && ok; ++sg) {
        int k;
        // (packed tiles; with several groups the panel segments come first: they are as wide as the tile and the first
        // product of a tile is the one that overwrites the accumulator)
        const int n_panel = tl.np - j_in;
        const bool diag_seg = pg ? sg >= n_panel : sg == 0;
        if (pg) {
          k = diag_seg ? tl.j + sg - n_panel : tl.i + sg;
          if (!diag_seg && j_in && k >= tl.j) ++k;   // skip type j: its rows have their one product already
        } else if (packed) {
          k = sg == 0 ? tl.j : tl.i + sg - 1;
          if (sg > 0 && j_in && k >= tl.j) ++k;   // skip type j: its rows have their one product already
        } else if (gp) {
          k = sg == 0 ? tl.i : tl.j + sg - 1;
          if (sg > 0 && i_in && k >= tl.i) ++k;   // group i: the panel product already holds x_i W_ii
        } else {
          k = n_seg == 1 ? tl.i : (sg == 0 ? min(tl.i, tl.j) : max(tl.i, tl.j));
        }
        for (int kb = 0; kb < nkb_seg; ++kb) {
          ok = __all_sync(0xffffffffu, wait_bar(empty0 + 8u * (uint32_t)stage, phase ^ 1u, ctl, a.status));
          if (!ok) break;
          const uint32_t bar = full0 + 8u * (uint32_t)stage;
          const uint32_t sa = smem0 + (uint32_t)stage * (uint32_t)C::kStageBytes;
          if (elect_one()) {
            if (loads_a && packed) {
              if (diag_seg) {   // all rows of the tile: np types x rows_per_type rows, type-major
                const int goff = (k - tl.j) * a.r;   // (with several groups only the 64-column boxes of group k are fetched)
                const int nb = pg ? (goff + a.r - 1) / 64 - goff / 64 + 1 : b_chunks;
                mbar_expect_tx(bar, (uint32_t)(a.pack * a.rows_per_type * BK * 2 + nb * C::kBChunkBytes));
                tma_load_4d(sa, &tmA, bar, kb * BK, k, 0, tl.i);
              } else {         // the rows of type k where they sit in the tile, zeros everywhere else
                mbar_expect_tx(bar, (uint32_t)(128 * BK * 2 + b_chunks * C::kBChunkBytes));
                tma_load_4d(sa, &tmA2, bar, kb * BK, k, -(k - tl.i) * a.rows_per_type, k);
              }
            } else if (loads_a) {
              // (a diagonal segment of a multi-group tile fetches only the 64-column boxes its group touches)
              const int goff = (k - tl.j) * a.r;
              const int nb = gp && sg > 0 ? (goff + a.r - 1) / 64 - goff / 64 + 1 : b_chunks;
              mbar_expect_tx(bar, (uint32_t)(a.a_box_rows * BK * 2 + nb * C::kBChunkBytes));
              if (a.sched == 2) tma_load_4d(sa, &tmA, bar, kb * BK, k, tl.i, a_row);
              else tma_load_3d(sa, &tmA, bar, kb * BK, k, a_row);
            } else if (pg ? diag_seg : gp && sg > 0) {
              // W_kk at the columns of its group inside the tile, zeros in the rest of the boxes it touches: column
              // (64 c - offset of the group in the tile) of group k is out of range on both sides of the group
              const int goff = (k - tl.j) * a.r;
              for (int c = goff / 64; c <= (goff + a.r - 1) / 64; ++c)
                tma_load_4d(sa + C::kABytes + c * C::kBChunkBytes, &tmB2, bar, c * 64 - goff, k, kb * BK, k);
            } else {
              for (int c = 0; c < a.n_chunks; ++c)
                tma_load_3d(sa + C::kABytes + c * C::kBChunkBytes, &tmB, bar, tl.n0_w + c * 64, kb * BK, k);
              for (int c = 0; c < (a.gated_f ? a.n_chunks : 0); ++c)   // the matching up columns, behind the gate chunks
                tma_load_3d(sa + C::kABytes + (a.n_chunks + c) * C::kBChunkBytes, &tmB, bar, a.gated_f + tl.n0_w + c * 64, kb * BK, k);
            }
          }
          __syncwarp();
          if (++stage == C::kStages) stage = 0, phase ^= 1u;
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    int stage = 0, acc = 0;
    uint32_t phase = 0, acc_phase = 0;
    bool ok = true;
    const uint32_t full0 = smem_u32(&ctl->full[0]), empty0 = smem_u32(&ctl->empty[0]);
    const uint32_t tfull0 = smem_u32(&ctl->tmem_full[0]), tempty0 = smem_u32(&ctl->tmem_empty[0]);
    const uint64_t da0 = make_smem_desc(smem_u32(smem), 16, C::kSboK, C::kSwzK);
    const uint64_t db0 = make_smem_desc(smem_u32(smem) + C::kABytes, C::kBChunkBytes, 1024);
    // instruction descriptor: D = f32, A = B = bf16, A K-major, B MN-major, N = tile_n, M = 128
    const int mma_n = a.gated_f ? 2 * a.n_chunks * 64 : a.tile_n;   // gated: gate chunks and up chunks side by side
    const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(mma_n >> 3) << 17) |
                           ((uint32_t)(128 >> 4) << 24);
    for (int t = blockIdx.x; ok; t += gridDim.x) {
      const Tile tl = decode_tile(a, ctl, t);
      if (tl.row0 < 0) break;
      const int j_in_t = tl.ng == 1 && tl.j >= tl.i && tl.j < tl.i + tl.np ? 1 : 0;
      const bool pg = a.pack > 1 && a.gpack > 1;
      const int n_kb = (pg            ? tl.ng + tl.np - j_in_t
                        : a.pack > 1  ? 1 + tl.np - j_in_t
                        : a.gpack > 1 ? 1 + tl.ng - (tl.i >= tl.j && tl.i < tl.j + tl.ng ? 1 : 0)
                                      : (tl.i == tl.j ? 1 : 2)) *
                       nkb_seg;
      if (lane == 0) ALG_TRACE(1, 1);
      ok = __all_sync(0xffffffffu, wait_bar(tempty0 + 8u * (uint32_t)acc, acc_phase ^ 1u, ctl, a.status));
      if (!ok) break;
      if (lane == 0) ALG_TRACE(1, 2);
      tc_fence_after();
      const uint32_t d_tmem = tmem_base + (uint32_t)(acc * TILE_N);
      const bool gp = a.gpack > 1 && !pg;
      const int i_in = gp && tl.i >= tl.j && tl.i < tl.j + tl.ng ? 1 : 0;
      for (int kb = 0; kb < n_kb; ++kb) {
        ok = __all_sync(0xffffffffu, wait_bar(full0 + 8u * (uint32_t)stage, phase, ctl, a.status));
        if (!ok) break;
        if (kb == 0 && lane == 0) ALG_TRACE(1, 3);
        tc_fence_after();
        const uint64_t da = da0 + (uint64_t)((uint32_t)stage * (uint32_t)(C::kStageBytes >> 4));
        uint64_t db = db0 + (uint64_t)((uint32_t)stage * (uint32_t)(C::kStageBytes >> 4));
        uint32_t d_seg = d_tmem, idesc_seg = idesc;
        if ((gp && kb >= nkb_seg) || (pg && kb >= (tl.np - j_in_t) * nkb_seg)) {
          // diagonal segment of a multi-group tile: only the 64-column boxes its group touches were fetched; the
          // product covers exactly those accumulator columns (zeros outside the group add nothing)
          int k = pg ? tl.j + kb / nkb_seg - (tl.np - j_in_t) : tl.j + kb / nkb_seg - 1;
          if (!pg && i_in && k >= tl.i) ++k;
          const int goff = (k - tl.j) * a.r;
          const int c_lo = goff / 64, c_hi = (goff + a.r - 1) / 64;
          db += (uint64_t)(c_lo * (C::kBChunkBytes >> 4));
          d_seg += (uint32_t)(c_lo * 64);
          idesc_seg = (idesc & ~(0x3Fu << 17)) | ((uint32_t)(((c_hi - c_lo + 1) * 64) >> 3) << 17);
        }
        if (elect_one()) {
#pragma unroll
          for (int kk = 0; kk < BK / 16; ++kk)
            tc_mma_bf16(d_seg, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 128), idesc_seg, (kb | kk) ? 1u : 0u);
          tc_commit(empty0 + 8u * (uint32_t)stage);
        }
        __syncwarp();
        if (++stage == C::kStages) stage = 0, phase ^= 1u;
      }
      if (!ok) break;
      if (elect_one()) tc_commit(tfull0 + 8u * (uint32_t)acc);
      __syncwarp();
      if (lane == 0) ALG_TRACE(1, 4);
      if (++acc == 2) acc = 0, acc_phase ^= 1u;
    }
  } else {
    // ---------------- epilogue ----------------
    const int e = warp - 2;
    const int quad = warp & 3;
    const int half = e >> 2;
    int acc = 0;
    uint32_t acc_phase = 0;
    // bf16 results leave through a 2 KB staging buffer per warp, 16 rows x 128 bytes at a time: every lane
    // holds 64 columns of its own row (128 bytes); sixteen lanes write their rows (16-byte pieces
    // XOR-swizzled by the row, conflict-free both ways), then eight lanes together store one whole row
    // segment, so one store instruction covers 4 rows x 128 contiguous bytes -- full lines.  What bounds
    // the store path of an SM is the number of line requests, not their bytes: rows of 64 bytes (32
    // columns per pass) were measured at about half the store rate.
    const uint32_t buf0 = smem_u32(store_buf + e * kStoreBufBytes);
    const uint32_t wr_row = buf0 + (uint32_t)(lane & 15) * 128u;
    const uint32_t wr_sw = (uint32_t)(lane & 7);
    const int rd_r = lane >> 3, rd_p = lane & 7;     // row within a group of four, 16-byte piece of the row
    const bool store8 = (a.r_out & 7) != 0;
    for (int t = blockIdx.x;; t += gridDim.x) {
      const Tile tl = decode_tile(a, ctl, t);
      if (tl.row0 < 0) break;
      const int r = quad * 32 + lane;
      int64_t out_row = -1;
      if (r < tl.rows) {
        if (a.sched_out == 2 && a.pack > 1) {   // rows of a packed tile are type-major: type tl.i + r / rows_per_type
          const int ti = fast_div(r, a.rows_per_type, a.inv_rpt);
          out_row = (int64_t)(r - ti * a.rows_per_type) * q + tl.i + ti;
        } else if (a.sched_out == 2) out_row = (int64_t)(tl.row0 + r - tl.i * a.rows_per_type) * q + tl.i;
        else if (a.sched_out == 0 && a.perm) out_row = __ldg(a.perm + tl.row0 + r);
        else out_row = tl.row0 + r;
        if (out_row >= a.M) out_row = -1;
      }
      bool ok = wait_bar(smem_u32(&ctl->tmem_full[acc]), acc_phase, ctl, a.status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      if (e == 0 && lane == 0) ALG_TRACE(2, 1);
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * TILE_N);
      const int col_end = tl.n0 + tl.cols;
      // Tiles of this path have short reductions, so the epilogue is the longest chain of a tile: warps
      // whose 32 rows lie past the tile's last row do nothing.
      const int c_end = quad * 32 < tl.rows ? tl.cols : 0;
      if (a.gated_f) {
        // gate values sit in accumulator columns [0, cols), the matching up values n_chunks * 64 columns further;
        // silu(g) * u with sigmoid(g) = (1 + tanh(g / 2)) / 2, then the 32 x 32 chunk goes through the warp's
        // buffer as 64-byte rows (four lanes store one row segment, 8 rows per store instruction)
        const uint32_t buf0 = smem_u32(store_buf + e * kStoreBufBytes);
        const uint32_t my_row = buf0 + (uint32_t)lane * 64u;
        const uint32_t sw = (uint32_t)((lane >> 1) & 3);
        const int sub = lane >> 2, piece = lane & 3;
        const uint32_t rd_base = buf0 + (uint32_t)sub * 64u;
        const uint32_t up_off = (uint32_t)(a.n_chunks * 64);
        int64_t dst_row[4];
#pragma unroll
        for (int g = 0; g < 4; ++g) dst_row[g] = __shfl_sync(0xffffffffu, out_row, g * 8 + sub);
#pragma unroll 1
        for (int c0 = half * 32; c0 < c_end; c0 += 64) {
          uint32_t vg[32], vu[32];
          tc_ld_32x32(taddr + (uint32_t)c0, vg);
          tc_ld_32x32(taddr + up_off + (uint32_t)c0, vu);
          tc_wait_ld();
          const int col = tl.n0 + c0;
          uint32_t w[16];
#pragma unroll
          for (int x = 0; x < 16; ++x) {
            float o[2];
#pragma unroll
            for (int y = 0; y < 2; ++y) {
              const float g = __uint_as_float(vg[2 * x + y]);
              float th;
              asm("tanh.approx.f32 %0, %1;" : "=f"(th) : "f"(0.5f * g));
              o[y] = g * fmaf(0.5f, th, 0.5f) * __uint_as_float(vu[2 * x + y]);
            }
            __nv_bfloat162 pk = __floats2bfloat162_rn(o[0], o[1]);
            w[x] = *(uint32_t *)&pk;
          }
          __syncwarp();
#pragma unroll
          for (int g = 0; g < 4; ++g)
            asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(my_row + ((((uint32_t)g) ^ sw) << 4)), "r"(w[g * 4]),
                         "r"(w[g * 4 + 1]), "r"(w[g * 4 + 2]), "r"(w[g * 4 + 3])
                         : "memory");
          __syncwarp();
          const bool piece_ok = col + piece * 8 < col_end;
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            const int rr = g * 8 + sub;
            const uint32_t rsw = (uint32_t)((rr >> 1) & 3);
            uint4 val;
            asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];"
                         : "=r"(val.x), "=r"(val.y), "=r"(val.z), "=r"(val.w)
                         : "r"(rd_base + (uint32_t)g * 512u + ((((uint32_t)piece) ^ rsw) << 4)));
            if (dst_row[g] >= 0 && piece_ok) *(uint4 *)((__nv_bfloat16 *)a.Y + dst_row[g] * a.ldy + col + piece * 8) = val;
          }
        }
      } else if (a.y_bf16) {
        int64_t dst_row[8];   // rows this lane stores for: phase * 16 + g * 4 + rd_r
#pragma unroll
        for (int g = 0; g < 8; ++g) dst_row[g] = __shfl_sync(0xffffffffu, out_row, g * 4 + rd_r);
        // the two warps of a quadrant alternate over the 64-column chunks
#pragma unroll 1
        for (int c0 = half * 64; c0 < c_end; c0 += 128) {
          uint32_t v0[32], v1[32];
          const bool second = c0 + 32 < c_end;
          tc_ld_32x32(taddr + (uint32_t)c0, v0);
          if (second) tc_ld_32x32(taddr + (uint32_t)(c0 + 32), v1);
          tc_wait_ld();
          const int col = tl.n0 + c0;
          uint32_t w[32];
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            float f[32];
#pragma unroll
            for (int x = 0; x < 32; ++x) f[x] = __uint_as_float(hh ? v1[x] : v0[x]);
            if (a.bias) {
              const __nv_bfloat16 *b = (const __nv_bfloat16 *)a.bias + col + hh * 32;
#pragma unroll
              for (int x = 0; x < 32; ++x)
                if (col + hh * 32 + x < col_end) f[x] += __bfloat162float(__ldg(b + x));
            }
            if (a.act == ALG_ACT_GELU_ERF) {
#pragma unroll
              for (int x = 0; x < 32; x += 2) gelu_erf2(f[x], f[x + 1]);
            } else if (a.act == ALG_ACT_GELU_TANH) {
#pragma unroll
              for (int x = 0; x < 32; ++x) f[x] = gelu_tanh(f[x]);
            }
#pragma unroll
            for (int x = 0; x < 16; ++x) {
              __nv_bfloat162 pk = __floats2bfloat162_rn(f[2 * x], f[2 * x + 1]);
              w[hh * 16 + x] = *(uint32_t *)&pk;
            }
          }
          const bool piece_ok = col + rd_p * 8 < col_end;
#pragma unroll
          for (int ph = 0; ph < 2; ++ph) {
            __syncwarp();   // the previous rows have been read out of the buffer
            if ((lane >> 4) == ph) {
#pragma unroll
              for (int pc = 0; pc < 8; ++pc)
                asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(wr_row + ((((uint32_t)pc) ^ wr_sw) << 4)),
                             "r"(w[pc * 4]), "r"(w[pc * 4 + 1]), "r"(w[pc * 4 + 2]), "r"(w[pc * 4 + 3])
                             : "memory");
            }
            __syncwarp();
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              const int rr = g * 4 + rd_r;     // row of the 16 staged ones
              uint4 val;
              asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];"
                           : "=r"(val.x), "=r"(val.y), "=r"(val.z), "=r"(val.w)
                           : "r"(buf0 + (uint32_t)rr * 128u + ((((uint32_t)rd_p) ^ (uint32_t)(rr & 7)) << 4)));
              const int64_t dr = dst_row[ph * 4 + g];
              if (a.gpack > 1) {
                // the piece's 8 accumulator columns lie in one group of the tile: group gi, column cg of it
                const int tc = c0 + rd_p * 8, gi = fast_div(tc, a.r, a.inv_r), cg = tc - gi * a.r;
                __nv_bfloat16 *dst = (__nv_bfloat16 *)a.Y + dr * a.ldy + tl.n0 + gi * a.r_out + cg;
                const bool in_tile = dr >= 0 && gi < tl.ng;
                if (store8) {
                  if (in_tile && cg < a.r_out) *(uint2 *)dst = make_uint2(val.x, val.y);
                  if (in_tile && cg + 4 < a.r_out) *(uint2 *)(dst + 4) = make_uint2(val.z, val.w);
                } else if (in_tile && cg < a.r_out) {
                  *(uint4 *)dst = val;
                }
              } else if (store8) {   // output groups start on 8 bytes only: two 4-column pieces, each stored if it belongs to the tile
                __nv_bfloat16 *dst = (__nv_bfloat16 *)a.Y + dr * a.ldy + col + rd_p * 8;
                if (dr >= 0 && piece_ok) *(uint2 *)dst = make_uint2(val.x, val.y);
                if (dr >= 0 && col + rd_p * 8 + 4 < col_end) *(uint2 *)(dst + 4) = make_uint2(val.z, val.w);
              } else if (dr >= 0 && piece_ok) {
                *(uint4 *)((__nv_bfloat16 *)a.Y + dr * a.ldy + col + rd_p * 8) = val;
              }
            }
          }
        }
      } else {
        // fp32 results: every lane stores its own row segment
#pragma unroll 1
        for (int c0 = half * 32; c0 < c_end; c0 += 64) {
          uint32_t v[32];
          tc_ld_32x32(taddr + (uint32_t)c0, v);
          tc_wait_ld();
          const int col = tl.n0 + c0;
          float f[32];
#pragma unroll
          for (int x = 0; x < 32; ++x) f[x] = __uint_as_float(v[x]);
          if (a.bias) {
            const __nv_bfloat16 *b = (const __nv_bfloat16 *)a.bias + col;
#pragma unroll
            for (int x = 0; x < 32; ++x)
              if (col + x < col_end) f[x] += __bfloat162float(__ldg(b + x));
          }
          if (a.act == ALG_ACT_GELU_ERF) {
#pragma unroll
            for (int x = 0; x < 32; x += 2) gelu_erf2(f[x], f[x + 1]);
          } else if (a.act == ALG_ACT_GELU_TANH) {
#pragma unroll
            for (int x = 0; x < 32; ++x) f[x] = gelu_tanh(f[x]);
          }
          if (out_row >= 0 && a.gpack > 1) {
#pragma unroll
            for (int g = 0; g < 8; ++g) {   // four accumulator columns lie in one group of the tile
              const int tc = c0 + g * 4, gi = fast_div(tc, a.r, a.inv_r), cg = tc - gi * a.r;
              if (gi < tl.ng && cg < a.r_out)
                *(float4 *)((float *)a.Y + out_row * a.ldy + tl.n0 + gi * a.r_out + cg) = make_float4(f[g * 4], f[g * 4 + 1], f[g * 4 + 2], f[g * 4 + 3]);
            }
          } else if (out_row >= 0) {
            float *dst = (float *)a.Y + out_row * a.ldy + col;
#pragma unroll
            for (int g = 0; g < 8; ++g)
              if (col + g * 4 < col_end) ((float4 *)dst)[g] = make_float4(f[g * 4], f[g * 4 + 1], f[g * 4 + 2], f[g * 4 + 3]);
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&ctl->tmem_empty[acc]));
      if (e == 0 && lane == 0) ALG_TRACE(2, 2);
      if (++acc == 2) acc = 0, acc_phase ^= 1u;
    }
  }

  // ---------------- teardown ----------------
  __syncwarp();
  if (ctl->abort_flag) {
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000LL) {   // copies still in flight land before shared memory is released
    }
  }
  tc_fence_before();
  __syncthreads();
  ALG_TRACE_CTA(1, 0);
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)C::kTmemCols)
                 : "memory");
  }
}

template <int TILE_N, int BK>
cudaError_t launch_t(const BigArgs &a, int num_sms, cudaStream_t st) {
  using C = Cfg<TILE_N, BK>;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(proj_big_kernel<TILE_N, BK>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  static_assert(C::kSmemBytes <= 227 * 1024, "shared memory budget");
  CUtensorMap tmA, tmA2, tmB;
  cudaError_t e;
  const BigArgs &b = a;
  if (b.pack > 1) {
    // X as {k in group, group, row in type, type}: interval rows of a type are consecutive, cyclic ones q apart
    const uint64_t rpt = (uint64_t)a.rows_per_type;
    const uint64_t dims[4] = {(uint64_t)a.s, (uint64_t)a.q, rpt, (uint64_t)a.q};
    const uint64_t str_i[3] = {(uint64_t)a.s * 2, (uint64_t)a.ldx * 2, (uint64_t)a.ldx * 2 * rpt};
    const uint64_t str_c[3] = {(uint64_t)a.s * 2, (uint64_t)a.ldx * 2 * (uint64_t)a.q, (uint64_t)a.ldx * 2};
    const uint32_t box_d[4] = {(uint32_t)BK, 1, (uint32_t)a.rows_per_type, (uint32_t)b.pack};
    const uint32_t box_p[4] = {(uint32_t)BK, 1, 128, 1};
    e = make_map_nd(&tmA, a.X, 4, dims, a.sched == 2 ? str_c : str_i, box_d, BK * 2);
    if (e == cudaSuccess) e = make_map_nd(&tmA2, a.X, 4, dims, a.sched == 2 ? str_c : str_i, box_p, BK * 2);
  } else if (a.sched == 2) {
    // rows of type i are rows i, i + q, ...: {k in group, group, type, position in the type}
    const uint64_t dims[4] = {(uint64_t)a.s, (uint64_t)a.q, (uint64_t)a.q, (uint64_t)a.rows_per_type};
    const uint64_t str[3] = {(uint64_t)a.s * 2, (uint64_t)a.ldx * 2, (uint64_t)a.ldx * 2 * (uint64_t)a.q};
    const uint32_t box[4] = {(uint32_t)BK, 1, 1, (uint32_t)a.a_box_rows};
    e = make_map_nd(&tmA, a.X, 4, dims, str, box, BK * 2);
  } else {
    const uint64_t dims[3] = {(uint64_t)a.s, (uint64_t)a.q, (uint64_t)a.M};
    const uint64_t str[2] = {(uint64_t)a.s * 2, (uint64_t)a.ldx * 2};
    const uint32_t box[3] = {(uint32_t)BK, 1, (uint32_t)a.a_box_rows};
    e = make_map_nd(&tmA, a.X, 3, dims, str, box, BK * 2);
  }
  if (e != cudaSuccess) return e;
  if (b.pack <= 1) tmA2 = tmA;
  CUtensorMap tmB2;
  if (b.gpack > 1) {
    // the bank by {column in group, column group, k in group, row group}
    const uint64_t dims[4] = {(uint64_t)a.r, (uint64_t)a.q, (uint64_t)a.s, (uint64_t)a.q};
    const uint64_t str[3] = {(uint64_t)a.r * 2, (uint64_t)a.ldw * 2, (uint64_t)a.ldw * 2 * (uint64_t)a.s};
    const uint32_t box[4] = {64, 1, (uint32_t)BK, 1};
    e = make_map_nd(&tmB2, a.W, 4, dims, str, box, 128);
    if (e != cudaSuccess) return e;
  }
  {
    // the bank as {columns, k in group, group}: rows past the group's width read as zero
    const uint64_t dims[3] = {(uint64_t)a.q * (uint64_t)a.r * (a.gated_f ? 2 : 1), (uint64_t)a.s, (uint64_t)a.q};
    const uint64_t str[2] = {(uint64_t)a.ldw * 2, (uint64_t)a.ldw * 2 * (uint64_t)a.s};
    const uint32_t box[3] = {64, (uint32_t)BK, 1};
    e = make_map_nd(&tmB, a.W, 3, dims, str, box, 128);
  }
  if (e != cudaSuccess) return e;
  long long tiles;
  if (b.pack > 1 && b.gpack > 1) {
    tiles = 0;
    const int g = b.gpack, n_units = (a.q + g - 1) / g;
    for (int i0 = 0; i0 < a.q; i0 += b.pack) {
      const int np = std::min(b.pack, a.q - i0), ua = i0 / g, ub = (i0 + np - 1) / g;
      tiles += n_units - (ub - ua + 1) + (std::min(a.q, (ub + 1) * g) - ua * g);
    }
  } else if (b.pack > 1) tiles = (long long)((a.q + b.pack - 1) / b.pack) * a.q * a.nt_n;
  else if (a.sched != 0) tiles = (long long)a.q * ((a.rows_per_type + 127) / 128) * b.col_units;
  else tiles = ((long long)a.M / 128 + a.q) * b.col_units;   // upper bound: every type may end in a ragged tile
  if (tiles >= (1ll << 31)) return cudaErrorInvalidValue;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)std::min<long long>(num_sms, std::max<long long>(tiles, 1)), 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = C::kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  if (b.gpack <= 1) tmB2 = tmB;
  e = cudaLaunchKernelEx(&cfg, proj_big_kernel<TILE_N, BK>, tmA, tmA2, tmB, tmB2, b);
  count_launch(1);
  return e;
}

}  // namespace

cudaError_t launch_proj_big(const BigArgs &in, int num_sms, cudaStream_t st) {
  cudaError_t e = tc_init();
  if (e != cudaSuccess) return e;
  BigArgs a = in;
  if ((a.sched == 0) != (a.sched_out == 0)) return cudaErrorInvalidValue;   // counted buckets on both sides or on neither
  if (a.q < 1 || a.q > kBigMaxQ || a.s % 8 || a.r % 8 || a.tile_n % 16 || a.tile_n < 16 || a.tile_n > 256) return cudaErrorInvalidValue;
  if (a.r_out % 4 || a.r_out < 4 || a.r_out > a.r) return cudaErrorInvalidValue;
  if (a.nt_n != (a.r_out + a.tile_n - 1) / a.tile_n || a.n_chunks != (a.tile_n + 63) / 64) return cudaErrorInvalidValue;
  if (a.a_box_rows < 8 || a.a_box_rows > 128 || a.a_box_rows % 8) return cudaErrorInvalidValue;
  // several row types per tile when a type fills at most half of one (equal buckets only)
  a.pack = a.sched != 0 && a.rows_per_type <= 64 ? std::min(a.q, 128 / a.rows_per_type) : 1;
  // several whole output groups per tile when they are narrow (one type per tile, no bias, no gate).  Measured:
  // 25600 -> 5120 at M = 32768: q = 64 (groups of 80) 0.557 -> 0.533 ms, q = 256 (24) 1.97 -> 1.57 ms; 5120 -> 25600 at
  // q = 256 (104) 1.49 -> 1.39 ms; groups of 128 lose (square product n = 8192: 0.065 -> 0.088 ms) and stay one per tile
  a.gpack = 1;
  a.col_units = a.q * a.nt_n;
  if (a.nt_n == 1 && !a.gated_f && !a.bias && a.r <= 112 && a.q >= 2) {
    // ... as many as keep at least four tiles per SM (2048 -> 768 in 16 groups of 48 at M = 2048 has 256 tiles of one
    // group: five groups per tile would leave 64 tiles for 148 SMs).  Together with several types per tile: a tile of
    // np types and ng groups runs np panel segments and ng diagonal segments instead of ng x (np + 1)
    // (25600 -> 5120 at q = 256, M = 2048: 34 segments per 24 columns before)
    const long long m_tiles = a.pack > 1    ? (a.q + a.pack - 1) / a.pack
                              : a.sched != 0 ? (long long)a.q * ((a.rows_per_type + 127) / 128)
                                             : std::max<long long>(a.q, a.M / 128);
    int g = std::min(a.q, 256 / a.r);
    while (g > 1 && m_tiles * ((a.q + g - 1) / g) < 4ll * num_sms) --g;
    if (g > 1) {
      a.gpack = g;
      a.col_units = (a.q + g - 1) / g;
      a.tile_n = (g * a.r + 15) / 16 * 16;
      a.n_chunks = (a.tile_n + 63) / 64;
    }
  }
  {
    const long long per = a.pack > 1 ? (long long)a.q * a.nt_n : a.sched != 0 ? (long long)((a.rows_per_type + 127) / 128) * a.col_units : 0;
    const long long total = a.pack > 1 ? per * ((a.q + a.pack - 1) / a.pack) : per * a.q;
    a.inv_per_type = per > 0 && total < (1 << 22) ? 1.f / (float)per : 0.f;
    a.inv_r = 1.f / (float)a.r;
    a.inv_g = 1.f / (float)a.gpack;
    a.inv_rpt = a.rows_per_type > 0 ? 1.f / (float)a.rows_per_type : 0.f;
    a.n_tg = (a.q + a.pack - 1) / a.pack;
    a.n_units = (a.q + a.gpack - 1) / a.gpack;
  }
  if (a.gated_f) {   // two accumulator halves of n_chunks * 64 columns each
    if (a.tile_n > 128 || !a.y_bf16 || a.r != a.r_out || a.gated_f != a.q * a.r || a.bias || a.act) return cudaErrorInvalidValue;
    return a.block_k == 64 ? launch_t<256, 64>(a, num_sms, st) : launch_t<256, 32>(a, num_sms, st);
  }
  if (a.tile_n <= 128) return a.block_k == 64 ? launch_t<128, 64>(a, num_sms, st) : launch_t<128, 32>(a, num_sms, st);
  return a.block_k == 64 ? launch_t<256, 64>(a, num_sms, st) : launch_t<256, 32>(a, num_sms, st);
}

}  // namespace algproj
