// Shared declarations of the algproj CUDA library (host metadata, device tables, launchers).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "algproj.h"

namespace algproj {

constexpr int kMaxQ = ALG_MAX_Q;
constexpr int kMaxPairs = kMaxQ * kMaxQ;
constexpr int kMaxClasses = 2 * kMaxPairs;  // per pair: full-width tiles and the remainder tile
constexpr int kMaxBucketChunks = 256;  // CTAs of the bucketing kernels (each scans all histograms)
// rows per bucketing CTA: a multiple of 256 that keeps the chunk count <= kMaxBucketChunks
inline int bucket_chunk_rows(int64_t M) {
  int64_t iters = (M + 256 * kMaxBucketChunks - 1) / (256 * kMaxBucketChunks);
  return (int)(256 * (iters > 0 ? iters : 1));
}

// A tile class = all tiles of one (row type i, output group j) pair that have the same width: the
// full-width tiles of the group, or its single narrower remainder tile.  Everything here is known
// on the host; only the number of 128- or 256-row tiles of type i depends on the batch.
struct ClassRec {
  unsigned i : 5, j : 5;
  unsigned cols : 10;     // width of every tile of the class
  unsigned n_tiles : 12;  // tiles of this class per m-tile (wider groups are cut into several classes)
  int col0;               // absolute first column of the class's first tile
};
static_assert(sizeof(ClassRec) == 8 && kMaxQ <= 32, "ClassRec packs a type index into 5 bits");

// Interaction table of one projection as the kernels see it (device memory, owned by a handle).
struct DevTable {
  int q;
  int n_pairs;                 // (type i, output group j) pairs with a non-empty support set
  int so[kMaxQ + 1];           // prefix sums of the input group widths  (S_k = [so[k], so[k+1]))
  int ro[kMaxQ + 1];           // prefix sums of the output group widths (R_j = [ro[j], ro[j+1]))
  uint32_t keep[kMaxPairs];    // keep[i*q+j] bit k set  <=>  k in B(i,j)
  // Tile classes, sorted by cost = K length x tile width, most expensive first (see ClassRec).
  int n_classes;
  ClassRec cls[kMaxClasses];
};

// One output tile of the grouped GEMM: rows [row0, row0+rows) of the type-bucketed row order
// (all of one type), columns [n0, n0+cols) inside one output group.
struct TileRec {
  int row0;
  int rows;
  int pair;   // (i * q + j) | (columns of the tile << 16)
  int n0;     // absolute first column
};

// Fixed-size header at the start of every workspace.
struct WsHeader {
  int offsets[kMaxQ + 2];  // offsets[t] = first bucketed row of type t; [q] = first bad row; [q+1] = M
  // the same buckets with every bucket padded to a multiple of 64 rows (weight-gradient pass):
  // pad_offsets[t] = first padded row of type t, [q] = end of the last bucket
  int pad_offsets[kMaxQ + 1];
};
static_assert(kMaxQ + 2 + kMaxQ + 1 <= 72, "workspace header layout");
static_assert(sizeof(WsHeader) <= 512, "workspace header stays within its slot");

struct TileGeom {
  int tile_m;        // rows per tile (a power of two)
  int tile_m_log2;
};

struct BucketArgs {
  const int32_t *types;  // nullptr => cyclic (row mod q)
  int M;
  int q;
  int chunk_rows;        // bucket_chunk_rows(M)
  WsHeader *hdr;
  int *big_offsets = nullptr;   // q > kMaxQ: bucket offsets [q + 2] go here instead of hdr->offsets
  int *chunk_counts;     // [n_chunks][q+1]
  int *perm;             // [M] bucketed position -> original row
  int *status;           // device status word of the handle
  unsigned int *sync;    // two counters of the handle (zero between launches) for the one-kernel variant
  long long wait_limit;  // bound of its wait, in SM clock cycles
  // rows with an out-of-range type get their output row zero-filled here
  void *Y;
  int64_t ldy;
  int N;
  int y_elem_bytes;
};

cudaError_t launch_bucket(const BucketArgs &a, cudaStream_t st);
// Xb[d, 0:K] = X[perm[d], 0:K] (16-byte vectors; K*elem_bytes % 16 == 0)
cudaError_t launch_gather_rows(const void *X, int64_t ldx, const int *perm, int M, int K,
                               int elem_bytes, void *Xb, cudaStream_t st);
// Weight-gradient pass (bf16): bucketed copies with every bucket padded to a multiple of 64 rows, pad
// rows zero.  Gp[p, 0:N] = G[perm[..], 0:N] for the padded row p;  XpT[c, p] = X[perm[..], c]
// (transposed: K x m_pad, leading dimension m_pad).  m_pad >= padded total (hdr->pad_offsets[q]).
cudaError_t launch_gather_rows_padded(const void *G, int64_t ldg, const WsHeader *hdr, const int *perm, int q, int m_pad,
                                      int N, void *Gp, cudaStream_t st);
cudaError_t launch_gather_transpose_padded(const void *X, int64_t ldx, const WsHeader *hdr, const int *perm, int q,
                                           int m_pad, int K, void *XpT, cudaStream_t st);

// Interaction table of a small-q handle, carried by value in the kernel parameters so that a
// kernel prologue needs no global metadata load.
constexpr int kParamQ = 8;
struct SmallTable {
  int valid;                              // q <= kParamQ and n_classes <= 2 * kParamQ * kParamQ
  int so[kParamQ + 1];
  int ro[kParamQ + 1];
  uint32_t keep[kParamQ * kParamQ];
  ClassRec cls[2 * kParamQ * kParamQ];
};

struct ProjArgs {
  const DevTable *tab;
  const int *offsets;     // device bucket offsets [q+2]; nullptr with the cyclic schedule (equal buckets)
  int cyclic_rows;        // M/q when offsets == nullptr
  int n_classes;          // tab->n_classes (host copy, sizes the shared-memory tile map)
  SmallTable st;          // by-value copy of the table when it is small
  TileGeom geom;
  const void *X;          // SIMT: original rows (gathered through perm); tcgen05: bucketed copy
  int64_t ldx;
  const int *perm;        // output row scatter: bucketed -> original; nullptr = keep bucketed
  const int *in_perm;     // SIMT only: input row gather (nullptr = X already bucketed)
  const void *W;
  int64_t ldw;
  const void *bias;
  int act;
  void *Y;
  int64_t ldy;
  int y_bf16;
  int M;
  int K;
  int N;
  int q;
  int *status;
  // Cyclic schedule (type of row b = b mod q, M a multiple of q) needs no permutation: rows of
  // type i are rows i, i+q, ... .  a_cyclic_rows = M/q makes the A operand a type-strided view of
  // the original X (3-D tensor map); out_cyclic_rows = M/q makes the epilogue compute
  // original row = (bucketed row - i*M/q)*q + i.  0 = off.
  int a_cyclic_rows;
  int out_cyclic_rows;
  // Interval schedule with a period (type of row b = (b mod run_period) / run_rows, run_rows = run_period / q):
  // the rows of a type come in runs of run_rows consecutive rows, one run per period.  With run_rows > 0 the two
  // fields above still switch the in-place views on, but the A operand is fetched in 64-row boxes from the view
  // {K, row in run, type, period} (run_rows is a multiple of 64, so a box never leaves its run) and the epilogue
  // computes original row = period * run_period + i * run_rows + row in run.  0 = cyclic addressing.
  int run_rows;
  int run_period;
  int b_3d;               // B tensor map is the 3-D chunked view (one copy per stage)
  int a_box_256;          // A tensor map carries 256-row boxes (one-CTA kernel with 256-row tiles)
  // Gradient passes.  w_kmajor: W is used transposed (B operand K-major; dX = G W^T): the reduction
  // runs over the COLUMNS of W, the output columns are its rows.  dyn_so: the q+1 offsets of the
  // reduction segments come from device memory (padded row buckets; dW = X^T G reduces over rows).
  int w_kmajor;
  const int *dyn_so;
  // Weight-gradient pass with the cyclic schedule and M a multiple of 64 q: nothing is copied.  The reduction
  // segment of type t is rows t, t + q, ... of X and of G read in place (type-strided views); the A operand is
  // the X block as it lies in memory (features contiguous: MN-major A).  seg_rows = M / q; 0 = off.
  int seg_rows;
  // Gated (SwiGLU) up projection: W is the merged bank [W_gate | W_up] with 2 * gated_f columns, a
  // tile accumulates 128 gate columns and the matching 128 up columns side by side, the epilogue
  // stores silu(gate) * up; N = gated_f is the width of the output.  0 = ordinary projection.
  int gated_f;
  int block_k;            // reduction depth of one pipeline stage of the one-CTA kernel: 64 or 32
  int y_staged;           // 1: the epilogue transposes bf16 results through shared memory for coalesced stores
  // Cyclic schedule: the tile sequences of all workers depend only on (handle, M) and are planned
  // once on the host; worker w reads plan[1 + w * plan_stride .. + plan_rounds) (the last record of
  // every worker is the end marker).  plan[0] is a stamp {row0 = M, rows = plan_tag}: a kernel whose
  // launch names another (M, tag) than the device copy holds plans for itself instead.
  // nullptr: every CTA plans for itself.
  const TileRec *plan;
  int plan_stride, plan_rounds, plan_tag;
  long long wait_limit;   // bound of every device-side wait, in SM clock cycles
};

cudaError_t launch_proj_simt(const ProjArgs &a, bool in_bf16, cudaStream_t st);

// Large-algebra path: complete-graph law with q equal groups, q up to kBigMaxQ, group widths that
// need not be multiples of the tile (proj_big.cu).
constexpr int kBigMaxQ = ALG_MAX_Q_LARGE;
struct BigArgs {
  const void *X;          // bf16; sched 0: type-bucketed copy, else the caller's rows
  int64_t ldx;
  const void *W;          // bf16 K x N bank
  int64_t ldw;
  const void *bias;       // bf16[N] or nullptr
  int act;
  void *Y;
  int64_t ldy;
  int y_bf16;
  int M, q;
  int s, r;               // width of every input / output group as the operands hold them (multiples of 8)
  int r_out;              // width of an output group in Y (a multiple of 4; < r when W was repacked with padding)
  int tile_n;             // columns per tile: multiple of 16, <= 256
  int nt_n;               // column tiles per output group = ceil(r / tile_n)
  int block_k;            // 64 or 32: reduction depth of a pipeline stage
  int n_chunks;           // 64-column boxes of W fetched per stage = ceil(tile_n / 64)
  int a_box_rows;         // rows of X fetched per stage: 128, or fewer when no type has that many rows
  int gated_f;            // > 0: SwiGLU up projection over the merged bank [W_gate | W_up] (2 * gated_f columns): a tile
                          // accumulates its gate columns and, n_chunks * 64 accumulator columns further, the matching
                          // up columns; the epilogue stores silu(gate) * up (bf16).  tile_n <= 128.
  int gpack;              // set by the launcher: output groups per tile (> 1 for narrow groups: one panel product over
                          // all of the tile's columns, then one diagonal product per group); needs pack == 1
  int col_units;          // set by the launcher: tiles per (row type, m-tile) = q * nt_n, or ceil(q / gpack)
  int pack;               // set by the launcher: row types per tile (> 1 when a type has at most 64 rows; sched 1, 2)
  int sched;              // 0: buckets from `offsets` (+ `perm` for the output rows), 1: interval, 2: cyclic
  int sched_out;          // how the rows of Y are addressed (same codes); differs from sched inside an FFN, whose
                          // hidden state stays in bucketed (= interval) order between its two projections
  const int *offsets;     // sched 0: device bucket offsets [q + 1]
  const int *perm;        // sched 0: bucketed row -> output row (nullptr = identity)
  int rows_per_type;      // sched 1, 2: M / q
  float inv_per_type;     // reciprocal of the tiles per type (or per type group) for the tile decode; 0 = divide  (set by the launcher)
  float inv_r;            // 1 / r: group of an accumulator column in tiles of several groups                   (set by the launcher)
  float inv_g, inv_rpt;   // 1 / gpack, 1 / rows_per_type                                                          (set by the launcher)
  int n_tg, n_units;      // type groups ceil(q / pack), column units ceil(q / gpack)                              (set by the launcher)
  int *status;
  long long wait_limit;
};
cudaError_t launch_proj_big(const BigArgs &a, int num_sms, cudaStream_t st);
// dst[R, gc * c_pad + cc] = src[row(R), gc * c + cc] for cc < c, else 0 -- column groups of c elements widened to
// c_pad; with rs > 0 the rows are grouped too (rs -> rs_pad, the extra rows zero).  perm (optional) maps a
// destination row to its source row (rows without row groups only).  c, c_pad multiples of 4; bf16.
cudaError_t launch_pad_groups(const void *src, int64_t ld_src, const int *perm, int rows_src, int n_col_groups, int c, int c_pad,
                              int rs, int rs_pad, void *dst, cudaStream_t st);

// tcgen05 paths.  One-CTA kernel: 128-row tiles, tile_n in {128, 192, 256}.  CTA-pair kernel
// (cta_group::2): 256-row tiles, 256 columns wide with a 128-column remainder tile.
constexpr int kTcSeqCap = 224, kTc2SeqCap = 48;  // precomputed tile records per worker
constexpr int kTcTileM = 128;
constexpr int kTcBlockK = 64;
constexpr int kDefaultStageK = 64;   // stage depth of the one-CTA GEMM kernel unless a handle asks otherwise
constexpr int kTc2TileM = 256;
constexpr int kTc2TileN = 256;
cudaError_t launch_proj_tc(const ProjArgs &a, int tile_n, int num_sms, cudaStream_t st);
cudaError_t launch_proj_tc_gated(const ProjArgs &a, int num_sms, cudaStream_t st);  // 128 output columns per tile
cudaError_t launch_proj_tc2(const ProjArgs &a, int num_sms, cudaStream_t st);
int tc2_max_pairs(int num_sms);  // CTA pairs that can be co-resident (0 on failure)
constexpr int kMaxWorkers = 256;
cudaError_t tc_init();  // resolves the driver entry point for tensor-map encoding

// decode path (M <= 64)
constexpr int kDecodeMaxM = 64;
constexpr int kDecodeParamQ = 8;   // tables of up to this many groups travel by value in the kernel parameters
struct DecodePlan {
  int sn;            // strip width in columns (64 or 32)
  int splits;        // K splits = cluster size (1..8)
  int box_rows;      // rows per TMA box of the weight slice (divides every s[k] / splits, <= 256)
  int w_smem_bytes;  // worst-case weight slice of one CTA
  int x_smem_bytes;  // worst-case staged X slice
  int p_smem_bytes;  // partial sums
};
struct DecodeArgs {
  const DevTable *tab;
  const void *X;
  int64_t ldx;
  const int32_t *types;   // nullptr => cyclic (row mod q)
  int M;
  const void *W;
  int64_t ldw;
  const void *bias;
  int act;
  void *Y;
  int64_t ldy;
  int y_bf16;
  int K;
  int N;
  int splits;
  uint32_t inv_splits;    // ceil(2^32 / splits): x / splits = umulhi(x, inv_splits) for x < 2^29, splits > 1 (set by the launcher)
  int box_rows;
  int w_smem_bytes;
  int x_smem_bytes;
  int *status;
  long long wait_limit;   // bound of every device-side wait, in SM clock cycles
  int extra_expect_bytes; // test aid: bytes added to the weight barrier's expectation that never arrive
  int q;
  int small_q;            // q <= kDecodeParamQ: the table below is valid
  int so[kDecodeParamQ + 1];
  int ro[kDecodeParamQ + 1];
  uint32_t keep[kDecodeParamQ * kDecodeParamQ];
};
bool decode_plan(int q, const int *s, int K, int N, int num_sms, DecodePlan *plan);
cudaError_t launch_decode(const DecodeArgs &a, const DecodePlan &plan, cudaStream_t st);

// decode step of the whole FFN in one launch (ffn_decode.cu), M <= kFfnDecodeMaxM
constexpr int kFfnDecodeMaxM = 16;
struct FfnDecodePlan {
  int su, sd;          // columns of the hidden state / of the output one CTA owns (multiples of 8)
  int n_up, n_dn;      // CTAs with an up strip / a down strip
  int wd_bytes, wu_bytes, stage_bytes, p_bytes, ctl_bytes;  // shared-memory regions
};
struct FfnDecodeArgs {
  const void *X;          // [M][D] bf16, packed
  const int32_t *types;   // nullptr => cyclic (row mod q)
  int M;
  const void *W_up, *W_down;   // canonical banks, packed: [D][F] and [F][D]
  const void *b_up, *b_down;
  int act;
  void *H;                // [M][F] bf16 scratch in global memory
  void *Y;                // [M][D]
  int y_bf16;
  int D, F, q;
  int su, sd, n_up, n_dn;
  int off_wu, off_stage, off_p, off_ctl;   // shared-memory offsets (the W_down slice sits at 0)
  int kc_up, kc_dn, m_pad;                 // K-chunk lengths of the staged activations; staged rows (8 or 16)
  unsigned int *counters;                  // [0] producers arrived, [1] consumers past the wait; zero between launches
  int *status;
  long long wait_limit;
  int extra_expect_bytes;
  const DevTable *tab_up, *tab_dn;         // tables in device memory (q > kDecodeParamQ)
  int small_q;
  int so_d[kDecodeParamQ + 1], so_f[kDecodeParamQ + 1];
  uint32_t keep[kDecodeParamQ * kDecodeParamQ];
};
bool ffn_decode_plan(int q, const int *dw, const int *fw, int D, int F, int num_sms, FfnDecodePlan *plan);
cudaError_t launch_ffn_decode(const FfnDecodeArgs &a, const FfnDecodePlan &plan, cudaStream_t st);

// Decode step of a few rows (complete-graph law, equal groups) in one launch: projection, FFN or gated FFN
// (row_decode.cu).
constexpr int kRowDecodeMaxM = 8;
struct RowDecodeArgs {
  int mode;                 // 0 gated FFN, 1 FFN, 2 projection (W1, b1, act; F = its output width, D = its input width)
  int M;                    // rows, 1 .. kRowDecodeMaxM
  const void *X;            // [M][ldx] bf16
  int64_t ldx;
  const int32_t *types;     // the rows' types; nullptr => row m has type m mod q (cyclic schedule)
  const void *W1;           // [D][ldw1] bf16: W_up, the merged bank [W_gate | W_up] (2 F columns), or the projection's W
  int64_t ldw1;
  const void *W2;           // [F][ldw2] bf16: W_down
  int64_t ldw2;
  const void *b1, *b2;      // bf16 biases or nullptr (not gated)
  int act;                  // activation of phase 1 (not gated)
  void *H;                  // [M][F] bf16 scratch in global memory, 16-byte aligned (FFN modes)
  void *Y;                  // [M][ldy]: D columns (projection: F)
  int64_t ldy;
  int y_bf16;
  int D, F, q;
  int gs, gr;               // group widths D / q and F / q, and their reciprocals  (set by the launcher)
  float inv_gs, inv_gr;
  int pc1, pc2;             // columns of a warp's piece (8 or 16)                 (set by the launcher)
  int ks1, ks2;             // warps sharing the weight rows of a piece            (set by the launcher)
  int units1, units2;       // pieces x sharing warps                              (set by the launcher)
  unsigned int *counters;   // [0] CTAs that finished phase 1, [1] CTAs past the wait; zero between launches (FFN modes)
  int *status;
  long long wait_limit;
  int extra_arrivals;       // test hook: arrivals the wait between the phases expects beyond the grid's (never come)
};
bool row_decode_fits(int q, int D, int F);
cudaError_t launch_row_decode(const RowDecodeArgs &a, int num_sms, cudaStream_t st);

void count_launch(int n = 1);
int handle_device(alg_proj_t h);  // device the handle was created on (-1 for a null handle)

constexpr long long kDefaultWaitLimit = 4000000000LL;  // ~2 s at B200 clocks

__host__ __device__ inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

}  // namespace algproj
