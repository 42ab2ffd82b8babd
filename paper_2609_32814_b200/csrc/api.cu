// C-ABI entry points: handle creation (interaction-table expansion, kernel selection), argument
// validation, workspace layout and the launch sequence of one forward pass.
#include <algorithm>
#include <atomic>
#include <cstring>
#include <new>
#include <vector>

#include "common.cuh"

using namespace algproj;

namespace algproj {
static std::atomic<int64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }
}  // namespace algproj

// One cached cyclic-schedule plan: the tile sequences of all workers for one M (device copy, pinned
// staging copy, event that marks the upload done).
struct PlanSlot {
  TileRec *d = nullptr, *h = nullptr;
  cudaEvent_t copied = nullptr;
  int64_t M = -1;
  int tag = 0, rounds = 0;
  uint64_t last_use = 0;
};
constexpr int kPlanSlots = 4;

// Large-algebra path (proj_big.cu): complete-graph law, equal group widths, q up to kBigMaxQ.
struct BigPlan {
  bool on = false;
  bool only = false;      // the handle has no interaction table: created for the large-algebra kernel alone
  bool eligible = false;  // the handle's law, dtype and widths fit the large-algebra kernel (GEMM_KERNEL = 4 may select it)
  int s = 0, r = 0;       // width of every input / output group
  int s_pad = 0, r_pad = 0;   // the same rounded up to multiples of 8: what the tensor maps can address
  bool repack = false;    // widths that are multiples of 4 only: X and W are repacked with padded groups on every call
  int tile_n = 0, nt_n = 0, block_k = 0;
};

struct alg_proj_s {
  BigPlan big;
  int q = 0;
  int s[kMaxQ] = {0}, r[kMaxQ] = {0};
  int K = 0, N = 0;
  alg_dtype_t dtype = ALG_F32;
  alg_schedule_t sched = ALG_SCHED_EXPLICIT;
  DevTable tab;             // host copy
  DevTable *d_tab = nullptr;
  int *d_status = nullptr;  // owned unless `shared_status`; followed by the two counters of the bucketing kernel
  bool shared_status = false;
  bool tc_ok = false;
  bool pair_kernel = false; // cta_group::2 kernel (256-row tiles)
  int tile_n = 0;           // tensor-core tile width of the one-CTA kernel
  // one-CTA kernel with 256-row x 128-column tiles (two accumulators per tile): taken when every
  // row type has enough rows to fill such tiles.  Its tile classes (128 columns wide) live in
  // `tab_tall` when the regular tile width is not 128.
  bool gated = false;       // SwiGLU up projection over the merged [W_gate | W_up] bank (N = F, W has 2 F columns)
  bool w_kmajor = false;    // input-gradient pass: W (N x K here) is used transposed
  bool dyn_segments = false;  // weight-gradient pass: the reduction segments are the padded row buckets of the call
  bool tall_ok = false;
  DevTable tab_tall;
  DevTable *d_tab_tall = nullptr;
  int device = 0;
  int num_sms = 148;
  int n_workers = 1;        // persistent CTAs (or CTA pairs) of the tensor-core kernel
  bool decode_ok = false;   // the small-M weight-streaming kernel covers this shape
  DecodePlan decode = {};
  // options (alg_proj_set_option)
  int opt_kernel = 0, opt_tile_n = 0, opt_stage_k = 0;
  bool opt_w_packed = false;     // large-algebra handle with padded groups: W arrives packed (alg_proj_pack_weight)
  int opt_row_gather = 0;        // explicit types: 0 / 1 copy pass, 2 rows fetched by the GEMM's producer warps
  int64_t interval_period = 0;   // INTERVAL schedule of a table-driven handle: period of the typing (0 = the whole batch)
  int opt_small_m = 1;           // 0 prefill kernels only, 1 the library's choice, 2 weight-streaming kernels only, 3 the row kernel wherever it fits
  bool opt_host_plan = true;
  long long wait_limit = kDefaultWaitLimit;
  int test_extra_expect = 0;
  // cyclic schedule: per-worker tile sequences of the one-CTA kernel for the last few M, planned on the host
  PlanSlot plan[kPlanSlots];
  int plan_stride = 0;
  uint64_t plan_clock = 0;
};

struct alg_ffn_s {
  alg_proj_s up, down;
  int D = 0, F = 0;
  bool timing = false;       // record events between the kernels of each forward call
  cudaEvent_t ev[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};
  // decode step of the whole FFN in one launch (M <= kFfnDecodeMaxM)
  bool gated = false;        // SwiGLU: up = merged gate/up projection with silu(gate) * up epilogue
  bool fd_ok = false;
  bool rd_ok = false;        // decode step of one row in one launch (row_decode.cu): gated, or plain without fd_ok
  FfnDecodePlan fd = {};
  unsigned int *d_counters = nullptr;
};

// Both gradient maps of one forward projection (s[q] -> r[q]).
struct alg_proj_grad_s {
  alg_proj_s dx;   // G (M x N) -> dX (M x K): groups swapped, support transposed, W used transposed
  alg_proj_s dw;   // rows = the K input features typed by their group, reduction over the padded row buckets
  int q = 0, K = 0, N = 0;
  alg_schedule_t sched = ALG_SCHED_EXPLICIT;
  int *d_feat_offsets = nullptr;   // [q+2] offsets of the feature groups: the "row buckets" of the dW problem
};

namespace {

std::atomic<int> g_plan_tag{1};  // stamps of host-built plans, unique within the process

size_t align_up(size_t v, size_t a = 256) { return (v + a - 1) / a * a; }

bool use_tc(const alg_proj_s &p) { return p.dtype == ALG_BF16 && p.tc_ok; }
int tile_m_of(const alg_proj_s &p) { return !use_tc(p) ? 64 : p.pair_kernel ? kTc2TileM : kTcTileM; }
int tile_n_of(const alg_proj_s &p) { return !use_tc(p) ? 64 : p.pair_kernel ? kTc2TileN : p.tile_n; }
int elem_bytes(alg_dtype_t d) { return d == ALG_BF16 ? 2 : 4; }

// Tile classes of a projection for tiles `tn` columns wide, sorted by cost = K length x tile width,
// most expensive first (stable).
alg_status_t build_classes(const alg_proj_s &p, int tn, DevTable &tab) {
  const int q = p.q;
  struct Item { long long cost; ClassRec rec; };
  std::vector<Item> order;
  for (int pr = 0; pr < q * q; ++pr) {
    long long len = 0;
    for (int k = 0; k < q; ++k)
      if ((p.tab.keep[pr] >> k) & 1u) len += p.s[k];
    const int i = pr / q, j = pr % q, width = p.r[j];
    for (int t0 = 0; t0 < width / tn; t0 += 4095) {  // n_tiles has 12 bits
      const int nt = std::min(4095, width / tn - t0);
      order.push_back({len * tn, ClassRec{(unsigned)i, (unsigned)j, (unsigned)tn, (unsigned)nt, p.tab.ro[j] + t0 * tn}});
    }
    if (width % tn)
      order.push_back({len * (width % tn),
                       ClassRec{(unsigned)i, (unsigned)j, (unsigned)(width % tn), 1u, p.tab.ro[j] + (width / tn) * tn}});
  }
  if ((int)order.size() > kMaxClasses) return ALG_ERR_INVALID_ARG;
  std::stable_sort(order.begin(), order.end(), [](const Item &x, const Item &y) { return x.cost > y.cost; });
  tab.n_classes = (int)order.size();
  for (size_t e = 0; e < order.size(); ++e) tab.cls[e] = order[e].rec;
  tab.n_pairs = q * q;
  return ALG_OK;
}

// Kernel selection and the tile classes that follow from it.  Runs at handle creation and again
// when an option that changes the selection is set.
alg_status_t configure_kernels(alg_proj_s &p) {
  const int q = p.q;
  const alg_dtype_t dtype = p.dtype;
  // tensor-core eligibility: bf16, K groups in 64-steps, N groups in 128-steps
  p.tc_ok = dtype == ALG_BF16;
  bool all256 = true, all192 = true, all128 = true;
  for (int g = 0; g < q; ++g) {
    if (p.s[g] % kTcBlockK) p.tc_ok = false;
    if (p.r[g] % 256) all256 = false;
    if (p.r[g] % 192) all192 = false;
    if (p.r[g] % 128) all128 = false;
  }
  if (!all256 && !all192 && !all128) p.tc_ok = false;
  p.tile_n = all256 ? 256 : all192 ? 192 : 128;
  if ((p.opt_tile_n == 256 && all256) || (p.opt_tile_n == 192 && all192) || (p.opt_tile_n == 128 && all128))
    p.tile_n = p.opt_tile_n;
  else if (p.opt_tile_n != 0)
    return ALG_ERR_UNSUPPORTED_SHAPE;
  // CTA-pair kernel whenever every output group splits into 256-wide tiles plus a 128-wide rest
  // (measured: it wins only when every tile has a long K loop; short loops favour the one-CTA kernel)
  int min_klen = 1 << 30;
  for (int pr = 0; pr < q * q; ++pr) {
    int len = 0;
    for (int k = 0; k < q; ++k)
      if ((p.tab.keep[pr] >> k) & 1u) len += p.s[k];
    min_klen = std::min(min_klen, len);
  }
  p.pair_kernel = p.tc_ok && all128 && min_klen >= 4096;
  if (p.gated && !(p.tc_ok && all128)) {
    // hidden groups off the 128-column grid: only the large-algebra kernel has a gated form for them (the caller
    // checks that the handle fits it)
    p.tc_ok = false;
    p.pair_kernel = false;
  } else if (p.gated) {   // 128 output columns per tile (the MMA is 256 wide: gate and up halves)
    if (p.opt_kernel > 1 || (p.opt_tile_n != 0 && p.opt_tile_n != 128)) return ALG_ERR_UNSUPPORTED_SHAPE;
    p.tile_n = 128;
    p.pair_kernel = false;
  }
  if (p.w_kmajor || p.dyn_segments) p.pair_kernel = false;   // the gradient passes run on the one-CTA kernel
  if (p.sched == ALG_SCHED_INTERVAL) p.pair_kernel = false;  // runs of a type are read in place by the one-CTA kernel only
  if (p.opt_kernel == 1) p.pair_kernel = false;
  if (p.opt_kernel == 2) {
    if (!(p.tc_ok && all128)) return ALG_ERR_UNSUPPORTED_SHAPE;
    p.pair_kernel = true;
  }

  alg_status_t bs = build_classes(p, tile_n_of(p), p.tab);
  if (bs != ALG_OK) return bs;
  // 256-row tiles: one-CTA kernel, 128-column tiles must divide every output group, and wider
  // tiles (which reuse A as well) must not be available
  p.tall_ok = p.tc_ok && !p.pair_kernel && !p.gated && all128 && !all256 && p.opt_tile_n == 0 && p.opt_kernel != 1;
  if (p.opt_kernel == 3) {
    if (!(p.tc_ok && all128)) return ALG_ERR_UNSUPPORTED_SHAPE;
    p.pair_kernel = false;
    p.tall_ok = true;
  }
  if (p.tall_ok) {
    p.tab_tall = p.tab;
    bs = build_classes(p, 128, p.tab_tall);
    if (bs != ALG_OK) return bs;
  }

  return ALG_OK;
}

alg_status_t pick_workers(alg_proj_s &p) {
  if (use_tc(p)) {
    p.n_workers = p.pair_kernel ? tc2_max_pairs(p.num_sms) : std::min(p.num_sms, kMaxWorkers);
    if (p.n_workers < 1) return ALG_ERR_CUDA;
  }
  return ALG_OK;
}

// Tiling of the large-algebra kernel: as few column tiles per output group as 256-wide tiles allow, the
// tile just wide enough (multiple of 16); 64-deep stages when the group width is a multiple of 64.
void plan_big(alg_proj_s &p, int s, int r) {
  p.big.on = true;
  p.big.s = s, p.big.r = r;
  p.big.s_pad = (s + 7) / 8 * 8, p.big.r_pad = (r + 7) / 8 * 8;
  p.big.repack = s % 8 != 0 || r % 8 != 0;
  const int widest = p.gated ? 128 : 256;   // a gated tile holds its gate columns and as many up columns
  p.big.nt_n = (r + widest - 1) / widest;
  p.big.tile_n = ((r + p.big.nt_n - 1) / p.big.nt_n + 15) / 16 * 16;
  p.big.nt_n = (r + p.big.tile_n - 1) / p.big.tile_n;
  // 64-deep stages whatever the group width: the copy engine is bound by row requests, and a 128-byte row of
  // X costs one request whether or not part of it is zero fill
  p.big.block_k = 64;
}

// Handle of the large-algebra path only (q > kMaxQ or the interval schedule): no interaction table.
alg_status_t init_big(alg_proj_s &p, int q, int s, int r, alg_schedule_t sched) {
  p.q = q;
  p.dtype = ALG_BF16;
  p.sched = sched;
  p.K = q * s;
  p.N = q * r;
  plan_big(p, s, r);
  p.big.only = true;
  if (q <= kMaxQ)
    for (int g = 0; g < q; ++g) p.s[g] = s, p.r[g] = r;
  if (cudaGetDevice(&p.device) != cudaSuccess) return ALG_ERR_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, p.device) != cudaSuccess) return ALG_ERR_CUDA;
  p.num_sms = prop.multiProcessorCount;
  if (prop.major != 10) return ALG_ERR_UNSUPPORTED_SHAPE;
  if (cudaMalloc(&p.d_status, 4 * sizeof(int)) != cudaSuccess) return ALG_ERR_CUDA;
  if (cudaMemset(p.d_status, 0, 4 * sizeof(int)) != cudaSuccess) return ALG_ERR_CUDA;
  if (tc_init() != cudaSuccess) return ALG_ERR_CUDA;
  return ALG_OK;
}

alg_status_t init_proj(alg_proj_s &p, int q, const int32_t *in_w, const int32_t *out_w, alg_dtype_t dtype,
                       alg_table_t table, const uint8_t *custom, alg_schedule_t sched, int *shared_status,
                       bool gated = false, bool allow_big = false) {
  p.gated = gated;
  if (q < 1 || q > kBigMaxQ || !in_w || !out_w) return ALG_ERR_INVALID_ARG;
  if (sched != ALG_SCHED_EXPLICIT && sched != ALG_SCHED_CYCLIC && sched != ALG_SCHED_INTERVAL) return ALG_ERR_INVALID_ARG;
  // large-algebra path: Q_q law, bf16, equal widths in multiples of 8
  bool big_fits = allow_big && table == ALG_TABLE_QQ && dtype == ALG_BF16 && in_w[0] > 0 && out_w[0] > 0 &&
                  in_w[0] % 4 == 0 && out_w[0] % 4 == 0;
  for (int g = 1; g < q && big_fits; ++g) big_fits = in_w[g] == in_w[0] && out_w[g] == out_w[0];
  if (q > kMaxQ || (sched == ALG_SCHED_INTERVAL && big_fits)) {
    if (!big_fits || (int64_t)q * in_w[0] > (1 << 30) || (int64_t)q * out_w[0] > (1 << 30)) return ALG_ERR_UNSUPPORTED_SHAPE;
    return init_big(p, q, in_w[0], out_w[0], sched);
  }
  // (an INTERVAL handle that does not fit the large-algebra path is a table-driven one: checked below)
  if (dtype != ALG_F32 && dtype != ALG_BF16) return ALG_ERR_INVALID_ARG;
  if (table != ALG_TABLE_QQ && table != ALG_TABLE_DENSE && table != ALG_TABLE_CUSTOM && table != ALG_TABLE_Q2POW)
    return ALG_ERR_INVALID_ARG;
  if (table == ALG_TABLE_Q2POW && (q & (q - 1)) != 0) return ALG_ERR_INVALID_ARG;  // q must be a power of two
  if (table == ALG_TABLE_CUSTOM && !custom) return ALG_ERR_INVALID_ARG;
  p.q = q;
  p.dtype = dtype;
  p.sched = sched;
  std::memset(&p.tab, 0, sizeof(p.tab));
  p.tab.q = q;
  int64_t K = 0, N = 0;
  for (int g = 0; g < q; ++g) {
    if (in_w[g] <= 0 || out_w[g] <= 0) return ALG_ERR_INVALID_ARG;
    p.s[g] = in_w[g];
    p.r[g] = out_w[g];
    p.tab.so[g] = (int)K;
    p.tab.ro[g] = (int)N;
    K += in_w[g];
    N += out_w[g];
    if (K > (1 << 30) || N > (1 << 30)) return ALG_ERR_INVALID_ARG;
  }
  p.tab.so[q] = (int)K;
  p.tab.ro[q] = (int)N;
  p.K = (int)K;
  p.N = (int)N;
  // support sets B(i,j): Q_q keeps k in {i,j} (Eqs. typed-diag / typed-off)
  for (int i = 0; i < q; ++i)
    for (int j = 0; j < q; ++j) {
      uint32_t m = 0;
      for (int k = 0; k < q; ++k) {
        // Q2POW: bits where k differs from i, and bits where k differs from j, must not overlap
        bool keep = table == ALG_TABLE_DENSE   ? true
                    : table == ALG_TABLE_QQ    ? (k == i || k == j)
                    : table == ALG_TABLE_Q2POW ? (((k ^ i) & (k ^ j)) == 0)
                                               : custom[((size_t)i * q + j) * q + k] != 0;
        if (keep) m |= 1u << k;
      }
      if (m == 0) return ALG_ERR_INVALID_ARG;  // an output block nobody writes
      p.tab.keep[i * q + j] = m;
    }
  alg_status_t cs = configure_kernels(p);
  if (cs != ALG_OK) return cs;
  if (sched == ALG_SCHED_INTERVAL && !use_tc(p)) return ALG_ERR_UNSUPPORTED_SHAPE;
  if (gated && !p.tc_ok && !(big_fits && in_w[0] % 8 == 0 && out_w[0] % 8 == 0)) return ALG_ERR_UNSUPPORTED_SHAPE;
  if (big_fits) {
    plan_big(p, in_w[0], out_w[0]);
    p.big.eligible = true;
    p.big.on = !p.tc_ok;   // by default only for widths the table-driven tensor path does not take
  }

  if (cudaGetDevice(&p.device) != cudaSuccess) return ALG_ERR_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, p.device) != cudaSuccess) return ALG_ERR_CUDA;
  p.num_sms = prop.multiProcessorCount;
  if (prop.major != 10) return ALG_ERR_UNSUPPORTED_SHAPE;  // sm_100a code only
  if (cudaMalloc(&p.d_tab, sizeof(DevTable)) != cudaSuccess) return ALG_ERR_CUDA;
  if (cudaMemcpy(p.d_tab, &p.tab, sizeof(DevTable), cudaMemcpyHostToDevice) != cudaSuccess) return ALG_ERR_CUDA;
  if (cudaMalloc(&p.d_tab_tall, sizeof(DevTable)) != cudaSuccess) return ALG_ERR_CUDA;
  if (cudaMemcpy(p.d_tab_tall, &p.tab_tall, sizeof(DevTable), cudaMemcpyHostToDevice) != cudaSuccess) return ALG_ERR_CUDA;
  if (shared_status) {
    p.d_status = shared_status;
    p.shared_status = true;
  } else {
    if (cudaMalloc(&p.d_status, 4 * sizeof(int)) != cudaSuccess) return ALG_ERR_CUDA;
    if (cudaMemset(p.d_status, 0, 4 * sizeof(int)) != cudaSuccess) return ALG_ERR_CUDA;
  }
  if (use_tc(p) && tc_init() != cudaSuccess) return ALG_ERR_CUDA;
  alg_status_t ws = pick_workers(p);
  if (ws != ALG_OK) return ws;
  if (use_tc(p) && sched == ALG_SCHED_CYCLIC) {
    // plans of the one-CTA kernel (the CTA-pair kernel always plans for itself)
    p.plan_stride = kTcSeqCap;
    const size_t bytes = (1 + (size_t)std::min(p.num_sms, kMaxWorkers) * p.plan_stride) * sizeof(TileRec);
    for (PlanSlot &sl : p.plan) {
      if (cudaMalloc(&sl.d, bytes) != cudaSuccess) return ALG_ERR_CUDA;
      if (cudaMemset(sl.d, 0, sizeof(TileRec)) != cudaSuccess) return ALG_ERR_CUDA;  // stamp of no plan
      if (cudaMallocHost(&sl.h, bytes) != cudaSuccess) return ALG_ERR_CUDA;
      if (cudaEventCreateWithFlags(&sl.copied, cudaEventDisableTiming) != cudaSuccess) return ALG_ERR_CUDA;
    }
  }
  if (dtype == ALG_BF16 && !p.gated && !p.w_kmajor && !p.dyn_segments && sched != ALG_SCHED_INTERVAL) {
    p.decode_ok = decode_plan(q, p.s, p.K, p.N, p.num_sms, &p.decode);
    for (int g = 0; g < q && p.decode_ok; ++g)
      if (p.r[g] % p.decode.sn) p.decode_ok = false;
    // The weight-streaming kernel was built for a few groups; with many groups and a large bank the prefill kernels
    // are several times faster (4096 -> 12288 at q = 32: M = 2 74 against 16 us, M = 64 377 against 46 us)
    if (q > kDecodeParamQ && (int64_t)p.K * p.N > (int64_t)4 << 20) p.decode_ok = false;
  }
  return ALG_OK;
}

void free_proj(alg_proj_s &p) {
  for (PlanSlot &sl : p.plan) {
    if (sl.d) cudaFree(sl.d);
    if (sl.h) cudaFreeHost(sl.h);
    if (sl.copied) cudaEventDestroy(sl.copied);
    sl = PlanSlot();
  }
  if (p.d_tab) cudaFree(p.d_tab);
  if (p.d_tab_tall) cudaFree(p.d_tab_tall);
  p.d_tab_tall = nullptr;
  if (p.d_status && !p.shared_status) cudaFree(p.d_status);
  p.d_tab = nullptr;
  p.d_status = nullptr;
}

struct WsLayout {
  size_t hdr = 0, chunks = 0, perm = 0, xb = 0, h = 0, total = 0;
  size_t xp = 0, wp = 0;   // large-algebra path with widths that are multiples of 4 only: repacked X and W
};

// `second`: the down projection of an FFN (nullptr for a single projection).
WsLayout layout(const alg_proj_s &first, const alg_proj_s *second, int64_t M) {
  WsLayout L;
  size_t off = 0;
  L.hdr = off;
  off = align_up(off + std::max(sizeof(WsHeader), (size_t)(first.q + 2) * sizeof(int)));   // more than kMaxQ types: a plain offset array
  L.chunks = off;
  off = align_up(off + (size_t)kMaxBucketChunks * (first.q + 1) * sizeof(int));
  L.perm = off;
  off = align_up(off + (size_t)M * sizeof(int));
  if (use_tc(first) || first.big.on) {
    L.xb = off;
    off = align_up(off + (size_t)M * first.K * 2, 1024);
  }
  if (first.big.on && first.big.repack) {
    L.xp = off;
    off = align_up(off + (size_t)M * first.q * first.big.s_pad * 2, 1024);
    L.wp = off;
    off = align_up(off + (size_t)first.q * first.big.s_pad * first.q * first.big.r_pad * 2, 1024);
  }
  if (second) {
    L.h = off;
    off = align_up(off + (size_t)M * first.N * elem_bytes(first.dtype), 1024);
  }
  L.total = off;
  return L;
}

alg_status_t cuda_status(cudaError_t e) { return e == cudaSuccess ? ALG_OK : ALG_ERR_CUDA; }

// Reduction depth of a pipeline stage of the one-CTA GEMM kernel (the CTA-pair kernel has its own, 64).
int block_k_of(const alg_proj_s &p) { return p.pair_kernel ? kTcBlockK : p.opt_stage_k ? p.opt_stage_k : kDefaultStageK; }

// Tiling of one forward call on the tensor-core path.
struct TcChoice {
  int tile_m, tile_n;
  const DevTable *tab;   // host copy with the tile classes of this tiling
  const DevTable *d_tab;
};
// 256-row tiles pay when every row type fills several of them (a ragged last tile then wastes
// little); with explicit types the rows per type are not known on the host: assume an even mix.
TcChoice choose_tiling(const alg_proj_s &p, int64_t M) {
  if (p.tall_ok && (p.opt_kernel == 3 || M / p.q >= 1024)) return {256, 128, &p.tab_tall, p.d_tab_tall};
  return {tile_m_of(p), tile_n_of(p), &p.tab, p.d_tab};
}

// Host twin of the in-kernel tile enumeration for the cyclic schedule (equal buckets of M/q rows):
// cost-sorted classes, m-tile major inside a class, boustrophedon assignment of tile indices to
// workers.  The plans of the last few M are cached in device memory the handle owns.  A new plan is
// written to a pinned staging copy and uploaded on `st` without waiting: the kernel that follows on
// the same stream finds it there, and the stamp in front of the records names (M, tag), so a kernel
// never follows a plan other than the one its launch was given.  Returns nullptr -- the kernels then
// plan for themselves, with the same result -- while `st` is being captured (a captured launch must
// not depend on handle state that later calls rewrite), when every slot's last upload is still in
// flight, or when the sequences do not fit.
const PlanSlot *prepare_cyclic_plan(alg_proj_s &p, const TcChoice &tc, int64_t M, cudaStream_t st) {
  if (!p.opt_host_plan || p.pair_kernel || !p.plan[0].d) return nullptr;
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(st, &cap) != cudaSuccess || cap != cudaStreamCaptureStatusNone) return nullptr;
  ++p.plan_clock;
  for (PlanSlot &sl : p.plan)
    if (sl.M == M) {
      sl.last_use = p.plan_clock;
      if (sl.rounds <= 0) return nullptr;
      // the upload may have been enqueued on another stream: order this one behind it
      if (cudaEventQuery(sl.copied) != cudaSuccess && cudaStreamWaitEvent(st, sl.copied, 0) != cudaSuccess) return nullptr;
      return &sl;
    }
  PlanSlot *slot = nullptr;
  for (PlanSlot &sl : p.plan) {
    if (sl.M >= 0 && cudaEventQuery(sl.copied) != cudaSuccess) continue;  // its staging copy is still being read
    if (!slot || sl.last_use < slot->last_use) slot = &sl;
  }
  if (!slot) return nullptr;
  const DevTable &tab = *tc.tab;
  const int q = p.q, nc = tab.n_classes, tile_m = tc.tile_m, nw = p.n_workers, stride = p.plan_stride;
  const int bucket = (int)(M / q);
  const int m_tiles = (bucket + tile_m - 1) / tile_m;
  std::vector<long long> prefix(nc + 1, 0);
  for (int c = 0; c < nc; ++c) prefix[c + 1] = prefix[c] + (long long)m_tiles * tab.cls[c].n_tiles;
  const long long total = prefix[nc];
  const long long all_rounds = (total + nw - 1) / nw;
  slot->M = M;
  slot->last_use = p.plan_clock;
  slot->rounds = 0;
  if (all_rounds + 1 > stride) return nullptr;
  std::vector<int> nkb(q * q, 0);
  for (int pr = 0; pr < q * q; ++pr)
    for (int k = 0; k < q; ++k)
      if ((p.tab.keep[pr] >> k) & 1u) nkb[pr] += p.s[k] / block_k_of(p);
  auto snake = [&](long long round, int w) { return round * nw + ((round & 1) ? (nw - 1 - w) : w); };
  const int rounds = (int)all_rounds + 1;
  slot->tag = g_plan_tag.fetch_add(1, std::memory_order_relaxed);
  TileRec stamp;
  stamp.row0 = (int)M, stamp.rows = slot->tag, stamp.pair = rounds, stamp.n0 = nw;
  slot->h[0] = stamp;
  for (int w = 0; w < nw; ++w) {
    const int valid = all_rounds == 0 ? 0 : (int)all_rounds - 1 + (snake(all_rounds - 1, w) < total ? 1 : 0);
    for (int pos = 0; pos < rounds; ++pos) {
      TileRec rec;
      rec.row0 = -1, rec.rows = 0, rec.pair = 0, rec.n0 = 0;
      if (pos < valid) {
        const long long idx = snake(pos, w);
        int c = (int)(std::upper_bound(prefix.begin(), prefix.end(), idx) - prefix.begin()) - 1;
        const ClassRec &r = tab.cls[c];
        const int loc = (int)(idx - prefix[c]), ntl = (int)r.n_tiles, mt = loc / ntl, nt = loc - mt * ntl;
        rec.row0 = (int)r.i * bucket + mt * tile_m;
        rec.rows = std::min(tile_m, bucket - mt * tile_m) | (nkb[(int)r.i * q + (int)r.j] << 16);
        rec.pair = ((int)r.i * q + (int)r.j) | ((int)r.cols << 16);
        rec.n0 = r.col0 + nt * (int)r.cols;
      }
      slot->h[1 + (size_t)w * stride + pos] = rec;
    }
  }
  if (cudaMemcpyAsync(slot->d, slot->h, (1 + (size_t)nw * stride) * sizeof(TileRec), cudaMemcpyHostToDevice, st) !=
          cudaSuccess ||
      cudaEventRecord(slot->copied, st) != cudaSuccess) {
    slot->M = -1;
    return nullptr;
  }
  slot->rounds = rounds;
  return slot;
}

bool aligned16(const void *p) { return ((uintptr_t)p & 15u) == 0; }

// Counted buckets (explicit types, or cyclic with q not dividing M) on the large-algebra kernel: always when the
// handle has no other tensor-core kernel or asks for it; by the library's choice when the buckets are small
// (at most two 128-row tiles per type on average) -- there the table-driven kernel spends its time on tile
// records and half-empty tiles (4096 -> 12288 at q = 32, M = 2048: 95.7 -> 70.1 us; FFN 187.6 -> 139.0 us),
// while with large buckets its tuned main loop and epilogue win (q = 8, M = 16384 FFN: 125.9 against 138.3 us).
bool use_big_counted(const alg_proj_s &p, int64_t M) {
  if (p.big.repack) return false;
  return p.big.on || (p.big.eligible && p.opt_kernel == 0 && M <= 256 * (int64_t)p.q);
}
// Equal buckets (cyclic schedule, q | M): by the library's choice when a type has at most 128 rows -- the
// large-algebra kernel then packs several types into a tile (FFN 4096 -> 12288 -> 4096 at q = 32, M = 2048:
// 128.6 -> 71.1 us); with fuller buckets the table-driven kernel is faster (58.6 against 63.2 us on the q = 2
// FFN at M = 8192).
bool use_big_equal(const alg_proj_s &p, int64_t M) {
  if (p.big.repack) return false;
  return p.big.on || (p.big.eligible && p.opt_kernel == 0 && M <= 128 * (int64_t)p.q);
}


alg_status_t run_proj(alg_proj_s &p, const WsLayout &L, char *ws, const void *X, int64_t ldx,
                      bool x_bucketed, const void *W, int64_t ldw, const void *bias, alg_act_t act, void *Y,
                      int64_t ldy, alg_dtype_t y_dtype, bool y_bucketed, int64_t M, cudaStream_t st,
                      cudaEvent_t after_gather = nullptr, bool cyclic = false, int run_rows = 0, int64_t run_period = 0) {
  if (cyclic && !run_rows && use_big_equal(p, M)) {
    // equal buckets on the large-algebra kernel: the caller's rows are read / written in place (type-strided),
    // a bucketed operand or result is the interval layout
    BigArgs g;
    g.X = X, g.ldx = ldx;
    g.W = W, g.ldw = ldw;
    g.bias = bias;
    g.act = (int)act;
    g.Y = Y, g.ldy = ldy;
    g.y_bf16 = y_dtype == ALG_BF16;
    g.M = (int)M, g.q = p.q;
    g.s = p.big.s, g.r = p.big.r, g.r_out = p.big.r;
    g.tile_n = p.big.tile_n, g.nt_n = p.big.nt_n;
    g.block_k = p.opt_stage_k == 32 ? 32 : p.big.block_k;
    g.n_chunks = (g.tile_n + 63) / 64;
    g.rows_per_type = (int)(M / p.q);
    g.a_box_rows = (int)std::min<int64_t>(128, (g.rows_per_type + 7) / 8 * 8);
    g.pack = 1;
    g.gated_f = p.gated ? p.N : 0;
    g.sched = x_bucketed ? 1 : 2, g.sched_out = y_bucketed ? 1 : 2;
    g.offsets = nullptr, g.perm = nullptr;
    g.status = p.d_status;
    g.wait_limit = p.wait_limit;
    if (after_gather) cudaEventRecord(after_gather, st);
    return cuda_status(launch_proj_big(g, p.num_sms, st));
  }
  if (!cyclic && use_big_counted(p, M)) {
    // large-algebra kernel on counted buckets: X bucketed already or gathered here, rows of Y scattered back
    // through the permutation unless the caller keeps the bucketed order
    BigArgs g;
    g.X = X, g.ldx = ldx;
    if (!x_bucketed) {
      if (launch_gather_rows(X, ldx, (const int *)(ws + L.perm), (int)M, p.K, 2, ws + L.xb, st) != cudaSuccess) return ALG_ERR_CUDA;
      g.X = ws + L.xb, g.ldx = p.K;
    }
    if (after_gather) cudaEventRecord(after_gather, st);
    g.W = W, g.ldw = ldw;
    g.bias = bias;
    g.act = (int)act;
    g.Y = Y, g.ldy = ldy;
    g.y_bf16 = y_dtype == ALG_BF16;
    g.M = (int)M, g.q = p.q;
    g.s = p.big.s, g.r = p.big.r, g.r_out = p.big.r;
    g.tile_n = p.big.tile_n, g.nt_n = p.big.nt_n;
    g.block_k = p.opt_stage_k == 32 ? 32 : p.big.block_k;
    g.n_chunks = (g.tile_n + 63) / 64;
    g.a_box_rows = 128;
    g.pack = 1;
    g.gated_f = p.gated ? p.N : 0;
    g.sched = 0, g.sched_out = 0;
    g.offsets = (const int *)(ws + L.hdr);
    g.perm = y_bucketed ? nullptr : (const int *)(ws + L.perm);
    g.rows_per_type = 0;
    g.status = p.d_status;
    g.wait_limit = p.wait_limit;
    return cuda_status(launch_proj_big(g, p.num_sms, st));
  }
  ProjArgs a;
  const TcChoice tc = choose_tiling(p, M);
  const DevTable &tab = *tc.tab;
  a.tab = tc.d_tab;
  a.offsets = cyclic ? nullptr : ((const WsHeader *)(ws + L.hdr))->offsets;
  a.cyclic_rows = cyclic ? (int)(M / p.q) : 0;
  a.n_classes = tab.n_classes;
  a.st.valid = p.q <= kParamQ && tab.n_classes <= 2 * kParamQ * kParamQ;
  if (a.st.valid) {
    for (int e = 0; e <= p.q; ++e) a.st.so[e] = tab.so[e], a.st.ro[e] = tab.ro[e];
    for (int e = 0; e < p.q * p.q; ++e) a.st.keep[e] = tab.keep[e];
    for (int e = 0; e < tab.n_classes; ++e) a.st.cls[e] = tab.cls[e];
  }
  a.geom.tile_m = tc.tile_m;
  a.geom.tile_m_log2 = a.geom.tile_m == 256 ? 8 : a.geom.tile_m == 128 ? 7 : 6;
  a.q = p.q;
  a.perm = (y_bucketed || cyclic) ? nullptr : (const int *)(ws + L.perm);  // cyclic outputs are addressed by arithmetic
  a.W = W;
  a.ldw = ldw;
  a.bias = bias;
  a.act = (int)act;
  a.Y = Y;
  a.ldy = ldy;
  a.y_bf16 = y_dtype == ALG_BF16;
  a.M = (int)M;
  a.K = p.K;
  a.N = p.N;
  a.status = p.d_status;
  a.a_cyclic_rows = (cyclic && !x_bucketed) ? (int)(M / p.q) : 0;
  a.out_cyclic_rows = (cyclic && !y_bucketed) ? (int)(M / p.q) : 0;
  a.run_rows = run_rows, a.run_period = (int)run_period;
  a.b_3d = 0;
  a.a_box_256 = 0;
  a.gated_f = p.gated ? p.N : 0;
  a.w_kmajor = p.w_kmajor ? 1 : 0;
  a.dyn_so = nullptr;
  a.seg_rows = 0;
  a.block_k = block_k_of(p);
  a.y_staged = 0;
  a.plan = nullptr;
  a.plan_stride = a.plan_rounds = a.plan_tag = 0;
  a.wait_limit = p.wait_limit;
  if (cyclic) {
    if (const PlanSlot *sl = prepare_cyclic_plan(p, tc, M, st)) {
      a.plan = sl->d;
      a.plan_stride = p.plan_stride;
      a.plan_rounds = sl->rounds;
      a.plan_tag = sl->tag;
    }
  }
  if (use_tc(p)) {
    a.in_perm = nullptr;
    if (x_bucketed || cyclic) {
      a.X = X;
      a.ldx = ldx;
    } else if (p.opt_row_gather == 2 && !p.pair_kernel && !p.w_kmajor && !p.dyn_segments && block_k_of(p) == 64) {
      // explicit types: the producer warps of the one-CTA kernel fetch the rows of a tile through the permutation,
      // four per copy instruction; X is read in place and no bucketed copy is written.  An option, not the
      // default: the copy engine needs longer for gathered rows than for a box (reductions of 1024..2048 columns:
      // 10 % slower), and where short reductions hide that (256 columns: a projection alone gains 10-13 % on
      // L2-resident rows) the FFN step with its working set rotating through HBM measures even or 1-2 % slower
      a.X = X;
      a.ldx = ldx;
      a.in_perm = (const int *)(ws + L.perm);
    } else {
      // explicit types: one pass writes the type-bucketed copy of X the tiled loads then read.  (Having
      // the GEMM's producer warps fetch the rows through the permutation themselves, with 16-byte
      // asynchronous copies into the swizzled image, was measured slower: the up projection of the
      // q = 4, M = 16384 configuration took 49 us against 36 us + 9 us for the copy.)
      cudaError_t e = launch_gather_rows(X, ldx, (const int *)(ws + L.perm), (int)M, p.K, 2, ws + L.xb, st);
      if (e != cudaSuccess) return ALG_ERR_CUDA;
      a.X = ws + L.xb;
      a.ldx = p.K;
    }
    if (after_gather) cudaEventRecord(after_gather, st);
    if (p.gated) return cuda_status(launch_proj_tc_gated(a, p.n_workers, st));
    if (p.pair_kernel) return cuda_status(launch_proj_tc2(a, p.num_sms, st));
    return cuda_status(launch_proj_tc(a, tc.tile_n, p.n_workers, st));
  }
  if (p.gated) return ALG_ERR_UNSUPPORTED_SHAPE;
  if (after_gather) cudaEventRecord(after_gather, st);
  a.X = X;
  a.ldx = ldx;
  a.in_perm = x_bucketed ? nullptr : (const int *)(ws + L.perm);
  return cuda_status(launch_proj_simt(a, p.dtype == ALG_BF16, st));
}

// INTERVAL schedule of a table-driven handle: rows per run and period for a batch of M rows; false if the batch
// does not split into whole periods of q runs of a multiple of 64 rows.
bool interval_runs(const alg_proj_s &p, int64_t M, int *run_rows, int64_t *period) {
  const int64_t P = p.interval_period ? p.interval_period : M;
  if (P <= 0 || M % P || P % p.q || (P / p.q) % 64) return false;
  *run_rows = (int)(P / p.q), *period = P;
  return true;
}

bool use_decode(const alg_proj_s &p, int64_t M) { return p.decode_ok && p.opt_small_m != 0 && M <= kDecodeMaxM; }
// a few rows under the complete-graph law with equal groups: the one-launch FMA kernel of row_decode.cu
// Rows up to which the row kernel is the library's choice.  It reads the diagonal block and the panel block of every
// row (2 M segments; repeats come from L2) and runs at about 2.5 us + 0.65 us per MB read, so it wins while that stays
// below what the prefill kernels need for a handful of rows: measured break-even near 20 MB for a projection (15-19 us
// through bucketing, gather and the GEMM) and 45 MB for an FFN (27-37 us).  Handles with a weight-streaming kernel
// (few groups, small banks) keep that one: 768 -> 3072 at q = 2 takes 4.9 us there against 6.3 us here at M = 1.
int row_decode_rows(const alg_proj_s &p) {
  if (p.decode_ok) return 0;
  const double per_row = 4.0 * p.K * (double)p.N / p.q;   // bytes: two segments of K / q rows of the bank
  return (int)std::max(1.0, std::min((double)kRowDecodeMaxM, 20e6 / per_row));
}
int row_decode_rows_ffn(int q, int D, int F, bool gated) {
  const double per_row = 4.0 * (gated ? 3 : 2) * D * (double)F / q;
  return (int)std::max(1.0, std::min((double)kRowDecodeMaxM, 45e6 / per_row));
}
bool use_row_decode(const alg_proj_s &p, int64_t M) {
  return M >= 1 && M <= (p.opt_small_m == 3 ? kRowDecodeMaxM : row_decode_rows(p)) && p.opt_small_m != 0 && p.opt_small_m != 2 && p.dtype == ALG_BF16 && (p.big.eligible || p.big.only) && !p.big.repack && !p.gated &&
         !p.w_kmajor && !p.dyn_segments && p.sched != ALG_SCHED_INTERVAL && row_decode_fits(p.q, p.K, p.N);
}

// Forward call on the large-algebra path.  Equal buckets (cyclic or interval schedule, q | M) need no
// pre-kernel at all; explicit types (q <= kMaxQ) go through bucketing and the row gather first.
alg_status_t run_big(alg_proj_s &p, const WsLayout &L, char *ws, const void *X, int64_t ldx, const int32_t *types,
                     int64_t M, const void *W, int64_t ldw, const void *bias, alg_act_t act, void *Y, int64_t ldy,
                     alg_dtype_t y_dtype, cudaStream_t st) {
  BigArgs a;
  a.X = X, a.ldx = ldx;
  a.W = W, a.ldw = ldw;
  a.bias = bias;
  a.act = (int)act;
  a.Y = Y, a.ldy = ldy;
  a.y_bf16 = y_dtype == ALG_BF16;
  a.M = (int)M, a.q = p.q;
  a.s = p.big.s, a.r = p.big.r;
  a.r_out = p.big.r;
  a.tile_n = p.big.tile_n, a.nt_n = p.big.nt_n;
  a.block_k = p.opt_stage_k == 32 ? 32 : p.big.block_k;
  a.n_chunks = (a.tile_n + 63) / 64;
  a.a_box_rows = 128;
  a.pack = 1;
  a.gated_f = 0;
  a.offsets = nullptr, a.perm = nullptr;
  a.rows_per_type = 0;
  a.status = p.d_status;
  a.wait_limit = p.wait_limit;
  const bool equal = p.sched != ALG_SCHED_EXPLICIT && M % p.q == 0;
  if (equal) {
    a.sched = p.sched == ALG_SCHED_INTERVAL ? 1 : 2;
    a.rows_per_type = (int)(M / p.q);
    a.a_box_rows = (int)std::min<int64_t>(128, (a.rows_per_type + 7) / 8 * 8);   // no type has more rows than that
  } else {
    if (p.sched == ALG_SCHED_INTERVAL) return ALG_ERR_INVALID_ARG;   // needs q | M
    BucketArgs b;
    b.types = p.sched == ALG_SCHED_CYCLIC ? nullptr : types;
    b.M = (int)M;
    b.q = p.q;
    b.chunk_rows = bucket_chunk_rows(M);
    b.hdr = (WsHeader *)(ws + L.hdr);
    if (p.q > kMaxQ) b.big_offsets = (int *)(ws + L.hdr);
    b.chunk_counts = (int *)(ws + L.chunks);
    b.perm = (int *)(ws + L.perm);
    b.status = p.d_status;
    b.sync = (unsigned int *)(p.d_status + 2);
    b.wait_limit = p.wait_limit;
    b.Y = Y;
    b.ldy = ldy;
    b.N = p.N;
    b.y_elem_bytes = elem_bytes(y_dtype);
    if (launch_bucket(b, st) != cudaSuccess) return ALG_ERR_CUDA;
    a.sched = 0;
    if (!p.big.repack) {   // (the repacking pass below gathers the rows itself)
      if (launch_gather_rows(X, ldx, b.perm, (int)M, p.K, 2, ws + L.xb, st) != cudaSuccess) return ALG_ERR_CUDA;
      a.X = ws + L.xb, a.ldx = p.K;
    }
    a.offsets = (const int *)(ws + L.hdr);   // WsHeader starts with its offsets
    a.perm = b.perm;
  }
  if (p.big.repack) {
    // groups widened to multiples of 8 with zeros: X (through the row permutation when there is one, straight from
    // the caller's rows instead of the gathered copy) and the bank, both rewritten on every call
    const bool permuted = a.sched == 0;
    if (launch_pad_groups(X, ldx, permuted ? a.perm : nullptr, (int)M, p.q, p.big.s, p.big.s_pad, 0, 0, ws + L.xp, st) != cudaSuccess)
      return ALG_ERR_CUDA;
    if (!p.opt_w_packed &&
        launch_pad_groups(W, ldw, nullptr, p.K, p.q, p.big.r, p.big.r_pad, p.big.s, p.big.s_pad, ws + L.wp, st) != cudaSuccess)
      return ALG_ERR_CUDA;
    a.X = ws + L.xp, a.ldx = (int64_t)p.q * p.big.s_pad;
    a.W = p.opt_w_packed ? W : ws + L.wp, a.ldw = (int64_t)p.q * p.big.r_pad;
    a.s = p.big.s_pad, a.r = p.big.r_pad;
  }
  a.sched_out = a.sched;
  return cuda_status(launch_proj_big(a, p.num_sms, st));
}

alg_status_t run_decode(const alg_proj_s &p, const void *X, int64_t ldx, const int32_t *types, int64_t M,
                        const void *W, int64_t ldw, const void *bias, alg_act_t act, void *Y, int64_t ldy,
                        alg_dtype_t y_dtype, cudaStream_t st) {
  DecodeArgs d;
  d.tab = p.d_tab;
  d.X = X;
  d.ldx = ldx;
  d.types = p.sched == ALG_SCHED_CYCLIC ? nullptr : types;
  d.M = (int)M;
  d.W = W;
  d.ldw = ldw;
  d.bias = bias;
  d.act = (int)act;
  d.Y = Y;
  d.ldy = ldy;
  d.y_bf16 = y_dtype == ALG_BF16;
  d.K = p.K;
  d.N = p.N;
  d.splits = p.decode.splits;
  d.box_rows = p.decode.box_rows;
  d.w_smem_bytes = p.decode.w_smem_bytes;
  d.x_smem_bytes = p.decode.x_smem_bytes;
  d.status = p.d_status;
  d.wait_limit = p.wait_limit;
  d.extra_expect_bytes = p.test_extra_expect;
  d.q = p.q;
  d.small_q = p.q <= kDecodeParamQ;
  if (d.small_q) {
    for (int e = 0; e <= p.q; ++e) d.so[e] = p.tab.so[e], d.ro[e] = p.tab.ro[e];
    for (int e = 0; e < p.q * p.q; ++e) d.keep[e] = p.tab.keep[e];
  }
  return cuda_status(launch_decode(d, p.decode, st));
}

}  // namespace

extern "C" {

alg_status_t alg_proj_create(alg_proj_t *out, int q, const int32_t *in_widths, const int32_t *out_widths,
                             alg_dtype_t dtype, alg_table_t table, const uint8_t *custom_keep,
                             alg_schedule_t schedule) {
  if (!out) return ALG_ERR_INVALID_ARG;
  *out = nullptr;
  alg_proj_s *p = new (std::nothrow) alg_proj_s();
  if (!p) return ALG_ERR_INVALID_ARG;
  alg_status_t s = init_proj(*p, q, in_widths, out_widths, dtype, table, custom_keep, schedule, nullptr, false, true);
  if (s != ALG_OK) {
    free_proj(*p);
    delete p;
    return s;
  }
  *out = p;
  return ALG_OK;
}

alg_status_t alg_proj_destroy(alg_proj_t h) {
  if (!h) return ALG_ERR_INVALID_ARG;
  free_proj(*h);
  delete h;
  return ALG_OK;
}

static alg_status_t set_option(alg_proj_s &p, alg_option_t option, int64_t value) {
  const bool no_table = p.big.only;   // large-algebra handles have one kernel
  switch (option) {
    case ALG_OPT_GEMM_KERNEL:
    case ALG_OPT_TILE_N: {
      if (no_table) return value == 0 || (option == ALG_OPT_GEMM_KERNEL && value == 4) ? ALG_OK : ALG_ERR_UNSUPPORTED_SHAPE;
      if (option == ALG_OPT_GEMM_KERNEL && (value < 0 || value > 4)) return ALG_ERR_INVALID_ARG;
      if (option == ALG_OPT_GEMM_KERNEL && value == 4) {   // the large-algebra kernel, for handles that fit it
        if (!p.big.eligible) return ALG_ERR_UNSUPPORTED_SHAPE;
        p.big.on = true;
        return ALG_OK;
      }
      if (option == ALG_OPT_GEMM_KERNEL && p.big.eligible) p.big.on = !p.tc_ok;
      if (option == ALG_OPT_TILE_N && value != 0 && value != 128 && value != 192 && value != 256) return ALG_ERR_INVALID_ARG;
      const int old_kernel = p.opt_kernel, old_tile = p.opt_tile_n;
      (option == ALG_OPT_GEMM_KERNEL ? p.opt_kernel : p.opt_tile_n) = (int)value;
      alg_status_t s = configure_kernels(p);
      if (s == ALG_OK) s = pick_workers(p);
      if (s != ALG_OK) {  // refuse: restore the previous selection
        p.opt_kernel = old_kernel, p.opt_tile_n = old_tile;
        configure_kernels(p);
        pick_workers(p);
        return s;
      }
      for (PlanSlot &sl : p.plan) sl.M = -1;  // cached plans belong to the old tiling
      int dev = 0;
      if (cudaGetDevice(&dev) != cudaSuccess || dev != p.device) return ALG_ERR_INVALID_ARG;
      // the device copy of the table may still be read by kernels in flight
      if (cudaDeviceSynchronize() != cudaSuccess) return ALG_ERR_CUDA;
      if (cudaMemcpy(p.d_tab, &p.tab, sizeof(DevTable), cudaMemcpyHostToDevice) != cudaSuccess) return ALG_ERR_CUDA;
      return cuda_status(cudaMemcpy(p.d_tab_tall, &p.tab_tall, sizeof(DevTable), cudaMemcpyHostToDevice));
    }
    case ALG_OPT_STAGE_K:
      if (value != 0 && value != 32 && value != 64) return ALG_ERR_INVALID_ARG;
      if (value == 32 && p.sched == ALG_SCHED_INTERVAL && !no_table) return ALG_ERR_UNSUPPORTED_SHAPE;  // runs: 64-deep only
      p.opt_stage_k = (int)value;
      for (PlanSlot &sl : p.plan) sl.M = -1;  // cached plans count K blocks of the old depth
      return ALG_OK;
    case ALG_OPT_WEIGHT_PACKED:
      if (value != 0 && value != 1) return ALG_ERR_INVALID_ARG;
      if (value == 1 && !(p.big.on && p.big.repack)) return ALG_ERR_UNSUPPORTED_SHAPE;
      p.opt_w_packed = value == 1;
      return ALG_OK;
    case ALG_OPT_ROW_GATHER:
      if (value < 0 || value > 2) return ALG_ERR_INVALID_ARG;
      p.opt_row_gather = (int)value;
      return ALG_OK;
    case ALG_OPT_INTERVAL_PERIOD:
      if (value < 0 || value > (1 << 30)) return ALG_ERR_INVALID_ARG;
      if (p.sched != ALG_SCHED_INTERVAL || (no_table && value != 0)) return ALG_ERR_UNSUPPORTED_SHAPE;
      if (value % ((int64_t)64 * p.q)) return ALG_ERR_INVALID_ARG;   // q runs of a multiple of 64 rows
      p.interval_period = value;
      return ALG_OK;
    case ALG_OPT_SMALL_M_KERNEL:
      if (value < 0 || value > 3) return ALG_ERR_INVALID_ARG;
      p.opt_small_m = (int)value;
      return ALG_OK;
    case ALG_OPT_HOST_PLAN: p.opt_host_plan = value != 0; return ALG_OK;
    case ALG_OPT_WAIT_LIMIT_CYCLES:
      if (value < 1000) return ALG_ERR_INVALID_ARG;
      p.wait_limit = value;
      return ALG_OK;
    case ALG_OPT_TEST_STALL_BYTES:
      if (value < 0 || value > (1 << 20) || value % 16) return ALG_ERR_INVALID_ARG;
      p.test_extra_expect = (int)value;
      return ALG_OK;
  }
  return ALG_ERR_INVALID_ARG;
}

alg_status_t alg_proj_set_option(alg_proj_t h, alg_option_t option, int64_t value) {
  if (!h) return ALG_ERR_INVALID_ARG;
  return set_option(*h, option, value);
}

alg_status_t alg_ffn_set_option(alg_ffn_t h, alg_option_t option, int64_t value) {
  if (!h) return ALG_ERR_INVALID_ARG;
  alg_status_t s = set_option(h->up, option, value);
  if (s != ALG_OK) return s;
  return set_option(h->down, option, value);
}

alg_status_t alg_proj_packed_weight_bytes(alg_proj_t h, size_t *bytes) {
  if (!h || !bytes) return ALG_ERR_INVALID_ARG;
  *bytes = h->big.on && h->big.repack ? (size_t)h->q * h->big.s_pad * (size_t)h->q * h->big.r_pad * 2 : 0;
  return ALG_OK;
}

alg_status_t alg_proj_pack_weight(alg_proj_t h, const void *W, int64_t ldw, void *W_packed, size_t packed_bytes, void *stream) {
  if (!h || !W || !W_packed) return ALG_ERR_INVALID_ARG;
  if (!(h->big.on && h->big.repack)) return ALG_ERR_UNSUPPORTED_SHAPE;
  size_t need = 0;
  alg_proj_packed_weight_bytes(h, &need);
  if (packed_bytes < need) return ALG_ERR_WORKSPACE_TOO_SMALL;
  if (ldw < h->N || !aligned16(W_packed)) return ALG_ERR_INVALID_ARG;
  return cuda_status(launch_pad_groups(W, ldw, nullptr, h->K, h->q, h->big.r, h->big.r_pad, h->big.s, h->big.s_pad, W_packed,
                                       (cudaStream_t)stream));
}

alg_status_t alg_proj_workspace_bytes(alg_proj_t h, int64_t max_M, size_t *bytes) {
  if (!h || !bytes || max_M < 0 || max_M > (1 << 30)) return ALG_ERR_INVALID_ARG;
  *bytes = layout(*h, nullptr, max_M).total;
  return ALG_OK;
}

alg_status_t alg_proj_forward(alg_proj_t h, const void *X, int64_t ldx, const int32_t *types, int64_t M,
                              const void *W, int64_t ldw, const void *bias, alg_act_t act, void *Y, int64_t ldy,
                              alg_dtype_t y_dtype, void *workspace, size_t workspace_bytes, void *stream) {
  if (!h || M < 0 || M > (1 << 30)) return ALG_ERR_INVALID_ARG;
  if (M == 0) return ALG_OK;
  if (!X || !W || !Y || !workspace) return ALG_ERR_INVALID_ARG;
  if (h->sched == ALG_SCHED_EXPLICIT && !types) return ALG_ERR_INVALID_ARG;
  if (h->opt_w_packed) ldw = (int64_t)h->q * h->big.r_pad;   // the packed bank has its own leading dimension
  if (ldx < h->K || ldw < (h->w_kmajor ? h->K : h->N) || ldy < h->N) return ALG_ERR_INVALID_ARG;
  if (y_dtype != ALG_F32 && y_dtype != ALG_BF16) return ALG_ERR_INVALID_ARG;
  if ((int)act < 0 || (int)act > 2) return ALG_ERR_INVALID_ARG;
  if (((uintptr_t)workspace & 255u) != 0) return ALG_ERR_INVALID_ARG;
  if (h->dtype == ALG_BF16) {
    if (!aligned16(X) || !aligned16(W) || ldx % 8 || ldw % 8) return ALG_ERR_INVALID_ARG;
  }
  if (!aligned16(Y) || (ldy * elem_bytes(y_dtype)) % 16) return ALG_ERR_INVALID_ARG;
  const WsLayout L = layout(*h, nullptr, M);
  if (workspace_bytes < L.total) return ALG_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = (cudaStream_t)stream;
  char *ws = (char *)workspace;
  if (use_row_decode(*h, M) && (!bias || aligned16(bias))) {
    // one row: one launch of plain FMAs over the 2 / q of the bank the row's type needs
    RowDecodeArgs d = {};
    d.mode = 2;
    d.M = (int)M;
    d.X = X, d.ldx = ldx;
    d.types = h->sched == ALG_SCHED_CYCLIC ? nullptr : types;
    d.W1 = W, d.ldw1 = ldw;
    d.b1 = bias;
    d.act = (int)act;
    d.Y = Y, d.ldy = ldy;
    d.y_bf16 = y_dtype == ALG_BF16;
    d.D = h->K, d.F = h->N, d.q = h->q;
    d.status = h->d_status;
    d.wait_limit = h->wait_limit;
    return cuda_status(launch_row_decode(d, h->num_sms, st));
  }
  if (use_decode(*h, M)) return run_decode(*h, X, ldx, types, M, W, ldw, bias, act, Y, ldy, y_dtype, st);
  if (h->big.on || (h->sched == ALG_SCHED_EXPLICIT && use_big_counted(*h, M)) ||
      (h->sched == ALG_SCHED_CYCLIC && M % h->q == 0 && use_big_equal(*h, M)))
    return run_big(*h, L, ws, X, ldx, types, M, W, ldw, bias, act, Y, ldy, y_dtype, st);

  BucketArgs b;
  b.types = h->sched == ALG_SCHED_CYCLIC ? nullptr : types;
  b.M = (int)M;
  b.q = h->q;
  b.chunk_rows = bucket_chunk_rows(M);
  b.hdr = (WsHeader *)(ws + L.hdr);
  b.chunk_counts = (int *)(ws + L.chunks);
  b.perm = (int *)(ws + L.perm);
  b.status = h->d_status;
  b.sync = (unsigned int *)(h->d_status + 2);
  b.wait_limit = h->wait_limit;
  b.Y = Y;
  b.ldy = ldy;
  b.N = h->N;
  b.y_elem_bytes = elem_bytes(y_dtype);
  if (h->sched == ALG_SCHED_INTERVAL) {   // runs of a type read and written in place
    int run_rows = 0;
    int64_t period = 0;
    if (!interval_runs(*h, M, &run_rows, &period)) return ALG_ERR_INVALID_ARG;
    return run_proj(*h, L, ws, X, ldx, false, W, ldw, bias, act, Y, ldy, y_dtype, false, M, st, nullptr, true, run_rows, period);
  }
  // cyclic schedule with equal buckets: no counting, no permutation, no gather
  const bool cyc = h->sched == ALG_SCHED_CYCLIC && use_tc(*h) && M % h->q == 0;
  if (!cyc && launch_bucket(b, st) != cudaSuccess) return ALG_ERR_CUDA;
  return run_proj(*h, L, ws, X, ldx, false, W, ldw, bias, act, Y, ldy, y_dtype, false, M, st, nullptr, cyc);
}

alg_status_t alg_proj_host_workspace_bytes(alg_proj_t h, int64_t max_M, alg_dtype_t y_dtype, size_t *bytes) {
  if (!h || !bytes || max_M < 0 || max_M > (1 << 30)) return ALG_ERR_INVALID_ARG;
  if (y_dtype != ALG_F32 && y_dtype != ALG_BF16) return ALG_ERR_INVALID_ARG;
  const size_t dev = align_up(layout(*h, nullptr, max_M).total);
  *bytes = dev + align_up((size_t)max_M * h->K * elem_bytes(h->dtype)) + align_up((size_t)max_M * sizeof(int32_t)) +
           align_up((size_t)max_M * h->N * elem_bytes(y_dtype));
  return ALG_OK;
}

alg_status_t alg_proj_forward_host(alg_proj_t h, const void *X_host, const int32_t *types_host, int64_t M, const void *W,
                                   int64_t ldw, const void *bias, alg_act_t act, void *Y_host, alg_dtype_t y_dtype,
                                   void *workspace, size_t workspace_bytes, void *stream) {
  if (!h || M < 0 || M > (1 << 30)) return ALG_ERR_INVALID_ARG;
  if (M == 0) return ALG_OK;
  if (!X_host || !Y_host || !workspace) return ALG_ERR_INVALID_ARG;
  if (h->sched == ALG_SCHED_EXPLICIT && !types_host) return ALG_ERR_INVALID_ARG;
  size_t need = 0;
  alg_status_t s = alg_proj_host_workspace_bytes(h, M, y_dtype, &need);
  if (s != ALG_OK) return s;
  if (workspace_bytes < need) return ALG_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = (cudaStream_t)stream;
  char *ws = (char *)workspace;
  const size_t dev = align_up(layout(*h, nullptr, M).total);
  const size_t xb = (size_t)M * h->K * elem_bytes(h->dtype), tb = (size_t)M * sizeof(int32_t);
  const size_t yb = (size_t)M * h->N * elem_bytes(y_dtype);
  char *dX = ws + dev, *dT = dX + align_up(xb), *dY = dT + align_up(tb);
  if (cudaMemcpyAsync(dX, X_host, xb, cudaMemcpyHostToDevice, st) != cudaSuccess) return ALG_ERR_CUDA;
  if (types_host && cudaMemcpyAsync(dT, types_host, tb, cudaMemcpyHostToDevice, st) != cudaSuccess) return ALG_ERR_CUDA;
  s = alg_proj_forward(h, dX, h->K, types_host ? (const int32_t *)dT : nullptr, M, W, ldw, bias, act, dY, h->N, y_dtype, ws, dev,
                       st);
  if (s != ALG_OK) return s;
  return cuda_status(cudaMemcpyAsync(Y_host, dY, yb, cudaMemcpyDeviceToHost, st));
}

alg_status_t alg_proj_gemm_count(alg_proj_t h, int64_t *n) {
  if (!h || !n) return ALG_ERR_INVALID_ARG;
  int64_t c = 0;
  if (h->big.only) c = 2 * (int64_t)h->q * h->q - h->q;   // no table: Q_q law (Eq. q-rank)
  else for (int pr = 0; pr < h->q * h->q; ++pr) c += __builtin_popcount(h->tab.keep[pr]);
  *n = c;
  return ALG_OK;
}

alg_status_t alg_proj_macs(alg_proj_t h, const int64_t *rows_per_type, int64_t *macs) {
  if (!h || !rows_per_type || !macs) return ALG_ERR_INVALID_ARG;
  int64_t total = 0;
  if (h->big.only) {   // no table: one product on the diagonal, two elsewhere
    for (int i = 0; i < h->q; ++i) {
      if (rows_per_type[i] < 0) return ALG_ERR_INVALID_ARG;
      total += rows_per_type[i] * (2 * (int64_t)h->q - 1) * h->big.s * h->big.r;
    }
    *macs = total;
    return ALG_OK;
  }
  for (int i = 0; i < h->q; ++i) {
    if (rows_per_type[i] < 0) return ALG_ERR_INVALID_ARG;
    for (int j = 0; j < h->q; ++j)
      for (int k = 0; k < h->q; ++k)
        if ((h->tab.keep[i * h->q + j] >> k) & 1u) total += rows_per_type[i] * (int64_t)h->s[k] * h->r[j];
  }
  *macs = total;
  return ALG_OK;
}

alg_status_t alg_proj_kernel_path(alg_proj_t h, int64_t M, alg_path_t *path) {
  if (!h || !path || M < 0) return ALG_ERR_INVALID_ARG;
  *path = use_row_decode(*h, M) || use_decode(*h, M) ? ALG_PATH_DECODE : (use_tc(*h) || h->big.on) ? ALG_PATH_TCGEN05 : ALG_PATH_SIMT;
  return ALG_OK;
}

static alg_status_t read_status(int *d_status, void *stream, alg_status_t *status) {
  if (!status) return ALG_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  int v = 0;
  if (cudaStreamSynchronize(st) != cudaSuccess) return ALG_ERR_CUDA;
  if (cudaMemcpy(&v, d_status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return ALG_ERR_CUDA;
  // a launch that gave up may have left the bucketing counters behind the status word half way
  if (v != 0 && cudaMemset(d_status, 0, 4 * sizeof(int)) != cudaSuccess) return ALG_ERR_CUDA;
  *status = (alg_status_t)v;
  return ALG_OK;
}

alg_status_t alg_proj_last_status(alg_proj_t h, void *stream, alg_status_t *status) {
  if (!h) return ALG_ERR_INVALID_ARG;
  return read_status(h->d_status, stream, status);
}

// ---- gradient maps (Appendix "Vector-Jacobian Products") ------------------------------------------

static alg_status_t support_of(int q, alg_table_t table, const uint8_t *custom, std::vector<uint8_t> &keep) {
  if (q < 1 || q > kMaxQ) return ALG_ERR_INVALID_ARG;
  if (table == ALG_TABLE_Q2POW && (q & (q - 1)) != 0) return ALG_ERR_INVALID_ARG;
  if (table == ALG_TABLE_CUSTOM && !custom) return ALG_ERR_INVALID_ARG;
  keep.assign((size_t)q * q * q, 0);
  for (int i = 0; i < q; ++i)
    for (int j = 0; j < q; ++j)
      for (int k = 0; k < q; ++k)
        keep[((size_t)i * q + j) * q + k] = table == ALG_TABLE_DENSE   ? 1
                                            : table == ALG_TABLE_QQ    ? (k == i || k == j)
                                            : table == ALG_TABLE_Q2POW ? (((k ^ i) & (k ^ j)) == 0)
                                                                       : custom[((size_t)i * q + j) * q + k] != 0;
  return ALG_OK;
}

alg_status_t alg_proj_grad_create(alg_proj_grad_t *out, int q, const int32_t *in_widths, const int32_t *out_widths,
                                  alg_table_t table, const uint8_t *custom_keep, alg_schedule_t schedule) {
  if (!out) return ALG_ERR_INVALID_ARG;
  *out = nullptr;
  if (!in_widths || !out_widths) return ALG_ERR_INVALID_ARG;
  if (table != ALG_TABLE_QQ && table != ALG_TABLE_DENSE && table != ALG_TABLE_CUSTOM && table != ALG_TABLE_Q2POW)
    return ALG_ERR_INVALID_ARG;
  std::vector<uint8_t> keep;
  alg_status_t s = support_of(q, table, custom_keep, keep);
  if (s != ALG_OK) return s;
  // dX: type i, output group k (of X), reduction over the output groups j with k in B(i,j)
  // dW: "row type" = feature group k, output group j, reduction over the row types i with k in B(i,j)
  std::vector<uint8_t> keep_dx((size_t)q * q * q), keep_dw((size_t)q * q * q);
  for (int i = 0; i < q; ++i)
    for (int j = 0; j < q; ++j)
      for (int k = 0; k < q; ++k) {
        keep_dx[((size_t)i * q + k) * q + j] = keep[((size_t)i * q + j) * q + k];
        keep_dw[((size_t)k * q + j) * q + i] = keep[((size_t)i * q + j) * q + k];
      }
  alg_proj_grad_s *g = new (std::nothrow) alg_proj_grad_s();
  if (!g) return ALG_ERR_INVALID_ARG;
  g->q = q;
  g->sched = schedule;
  g->dx.w_kmajor = true;
  s = init_proj(g->dx, q, out_widths, in_widths, ALG_BF16, ALG_TABLE_CUSTOM, keep_dx.data(), schedule, nullptr);
  if (s == ALG_OK) {
    int32_t seg[kMaxQ];
    for (int e = 0; e < q; ++e) seg[e] = kTcBlockK;   // placeholders: the segments of a call are its padded row buckets
    g->dw.dyn_segments = true;
    s = init_proj(g->dw, q, seg, out_widths, ALG_BF16, ALG_TABLE_CUSTOM, keep_dw.data(), ALG_SCHED_EXPLICIT, g->dx.d_status);
    if (s == ALG_ERR_INVALID_ARG) s = ALG_ERR_UNSUPPORTED_SHAPE;   // a weight block no row type ever uses
  }
  if (s == ALG_OK && !(use_tc(g->dw) && g->dw.tc_ok)) s = ALG_ERR_UNSUPPORTED_SHAPE;   // dW has no SIMT path
  if (s == ALG_OK && g->dw.tile_n > 128) {
    // dW has as many tiles as the weight bank has 128 x tile_n blocks, whatever the batch: when wide tiles
    // leave SMs without work, 128-column tiles (twice as many) are the better trade
    long long tiles = 0;
    bool all128 = true;
    for (int e = 0; e < q; ++e) {
      tiles += (long long)((in_widths[e] + 127) / 128) * (g->dx.K / g->dw.tile_n);
      if (out_widths[e] % 128) all128 = false;
    }
    if (all128 && tiles < g->dw.num_sms) s = set_option(g->dw, ALG_OPT_TILE_N, 128);
  }
  if (s == ALG_OK) {
    g->K = g->dx.N, g->N = g->dx.K;
    int offs[kMaxQ + 2];
    for (int e = 0; e <= q; ++e) offs[e] = g->dx.tab.ro[e];   // feature-group offsets
    offs[q + 1] = g->K;
    if (cudaMalloc(&g->d_feat_offsets, (q + 2) * sizeof(int)) != cudaSuccess ||
        cudaMemcpy(g->d_feat_offsets, offs, (q + 2) * sizeof(int), cudaMemcpyHostToDevice) != cudaSuccess)
      s = ALG_ERR_CUDA;
  }
  if (s != ALG_OK) {
    if (g->d_feat_offsets) cudaFree(g->d_feat_offsets);
    free_proj(g->dw);
    free_proj(g->dx);
    delete g;
    return s;
  }
  *out = g;
  return ALG_OK;
}

alg_status_t alg_proj_grad_destroy(alg_proj_grad_t h) {
  if (!h) return ALG_ERR_INVALID_ARG;
  if (h->d_feat_offsets) cudaFree(h->d_feat_offsets);
  free_proj(h->dw);
  free_proj(h->dx);
  delete h;
  return ALG_OK;
}

namespace {
int padded_rows(const alg_proj_grad_s &g, int64_t M) { return (int)((M + 63) / 64 * 64) + 64 * g.q; }
struct GradLayout {
  size_t hdr, chunks, perm, xt, gp, total;
};
GradLayout grad_layout(const alg_proj_grad_s &g, int64_t M) {
  GradLayout L;
  size_t off = 0;
  L.hdr = off;
  off = align_up(off + sizeof(WsHeader));
  L.chunks = off;
  off = align_up(off + (size_t)kMaxBucketChunks * (g.q + 1) * sizeof(int));
  L.perm = off;
  off = align_up(off + (size_t)M * sizeof(int));
  const size_t mp = (size_t)padded_rows(g, M);
  L.xt = off;
  off = align_up(off + mp * g.K * 2, 1024);
  L.gp = off;
  off = align_up(off + mp * g.N * 2, 1024);
  L.total = off;
  return L;
}
}  // namespace

alg_status_t alg_proj_grad_workspace_bytes(alg_proj_grad_t h, int64_t max_M, size_t *bytes) {
  if (!h || !bytes || max_M < 0 || max_M > (1 << 30)) return ALG_ERR_INVALID_ARG;
  *bytes = std::max(layout(h->dx, nullptr, max_M).total, grad_layout(*h, max_M).total);
  return ALG_OK;
}

alg_status_t alg_proj_grad_input(alg_proj_grad_t h, const void *G, int64_t ldg, const int32_t *types, int64_t M,
                                 const void *W, int64_t ldw, void *dX, int64_t lddx, alg_dtype_t x_dtype, void *workspace,
                                 size_t workspace_bytes, void *stream) {
  if (!h) return ALG_ERR_INVALID_ARG;
  return alg_proj_forward(&h->dx, G, ldg, types, M, W, ldw, nullptr, ALG_ACT_NONE, dX, lddx, x_dtype, workspace,
                          workspace_bytes, stream);
}

alg_status_t alg_proj_grad_weight(alg_proj_grad_t h, const void *X, int64_t ldx, const void *G, int64_t ldg,
                                  const int32_t *types, int64_t M, void *dW, int64_t lddw, alg_dtype_t w_dtype,
                                  void *workspace, size_t workspace_bytes, void *stream) {
  if (!h || M < 0 || M > (1 << 30)) return ALG_ERR_INVALID_ARG;
  if (!X || !G || !dW || !workspace) return ALG_ERR_INVALID_ARG;
  if (h->sched == ALG_SCHED_EXPLICIT && !types && M > 0) return ALG_ERR_INVALID_ARG;
  if (ldx < h->K || ldg < h->N || lddw < h->N) return ALG_ERR_INVALID_ARG;
  if (w_dtype != ALG_F32 && w_dtype != ALG_BF16) return ALG_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(G) || !aligned16(dW) || ldx % 8 || ldg % 8 || (lddw * elem_bytes(w_dtype)) % 16)
    return ALG_ERR_INVALID_ARG;
  if (((uintptr_t)workspace & 255u) != 0) return ALG_ERR_INVALID_ARG;
  const GradLayout L = grad_layout(*h, M);
  if (workspace_bytes < L.total) return ALG_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = (cudaStream_t)stream;
  char *ws = (char *)workspace;
  alg_proj_s &p = h->dw;
  const int mp = padded_rows(*h, M);
  WsHeader *hdr = (WsHeader *)(ws + L.hdr);
  // Cyclic schedule with whole 64-row blocks per type: the buckets are rows t, t + q, ... of X and of G as they
  // lie in memory, nothing is counted, permuted, transposed or copied (the kernel reads both through
  // type-strided views and takes the X block as an MN-major A operand).
  const bool in_place = h->sched == ALG_SCHED_CYCLIC && M > 0 && M % (64 * (int64_t)h->q) == 0 && block_k_of(p) == 64;
  // 1. row buckets of this batch (also for the cyclic schedule: the copies below need the permutation)
  BucketArgs b;
  b.types = h->sched == ALG_SCHED_CYCLIC ? nullptr : types;
  b.M = (int)M;
  b.q = h->q;
  b.chunk_rows = bucket_chunk_rows(M);
  b.hdr = hdr;
  b.chunk_counts = (int *)(ws + L.chunks);
  b.perm = (int *)(ws + L.perm);
  b.status = p.d_status;
  b.sync = (unsigned int *)(p.d_status + 2);
  b.wait_limit = p.wait_limit;
  b.Y = nullptr;   // nothing to zero: a row with an out-of-range type simply contributes to no block
  b.ldy = 0, b.N = 0, b.y_elem_bytes = 0;
  if (M > 0 && !in_place && launch_bucket(b, st) != cudaSuccess) return ALG_ERR_CUDA;
  if (M == 0) {   // no rows: every block of dW is zero
    return cuda_status(cudaMemset2DAsync(dW, (size_t)lddw * elem_bytes(w_dtype), 0, (size_t)h->N * elem_bytes(w_dtype),
                                         (size_t)h->K, st));
  }
  // 2. padded, bucketed copies: X transposed (K x m_pad), G as it is (m_pad x N); pad rows are zero
  if (!in_place) {
    if (launch_gather_transpose_padded(X, ldx, hdr, b.perm, h->q, mp, h->K, ws + L.xt, st) != cudaSuccess) return ALG_ERR_CUDA;
    if (launch_gather_rows_padded(G, ldg, hdr, b.perm, h->q, mp, h->N, ws + L.gp, st) != cudaSuccess) return ALG_ERR_CUDA;
  }
  // 3. the grouped GEMM: rows = input features (type = their group), reduction over the padded buckets
  ProjArgs a;
  const TcChoice tc = {tile_m_of(p), tile_n_of(p), &p.tab, p.d_tab};
  const DevTable &tab = p.tab;
  a.tab = tc.d_tab;
  a.offsets = h->d_feat_offsets;
  a.cyclic_rows = 0;
  a.n_classes = tab.n_classes;
  a.st.valid = p.q <= kParamQ && tab.n_classes <= 2 * kParamQ * kParamQ;
  if (a.st.valid) {
    for (int e = 0; e <= p.q; ++e) a.st.so[e] = tab.so[e], a.st.ro[e] = tab.ro[e];
    for (int e = 0; e < p.q * p.q; ++e) a.st.keep[e] = tab.keep[e];
    for (int e = 0; e < tab.n_classes; ++e) a.st.cls[e] = tab.cls[e];
  }
  a.geom.tile_m = tc.tile_m;
  a.geom.tile_m_log2 = 7;
  a.q = p.q;
  a.perm = nullptr;
  a.in_perm = nullptr;
  a.X = in_place ? X : (const void *)(ws + L.xt);
  a.ldx = in_place ? ldx : mp;
  a.W = in_place ? G : (const void *)(ws + L.gp);
  a.ldw = in_place ? ldg : h->N;
  a.bias = nullptr;
  a.act = (int)ALG_ACT_NONE;
  a.Y = dW;
  a.ldy = lddw;
  a.y_bf16 = w_dtype == ALG_BF16;
  a.M = h->K;          // rows of this GEMM = input features
  a.K = in_place ? (int)M : mp;   // reduction = (padded) rows of the batch
  a.N = h->N;
  a.status = p.d_status;
  a.a_cyclic_rows = 0;
  a.out_cyclic_rows = 0;
  a.run_rows = 0, a.run_period = 0;
  a.b_3d = 0;
  a.a_box_256 = 0;
  a.gated_f = 0;
  a.w_kmajor = 0;
  a.dyn_so = in_place ? nullptr : hdr->pad_offsets;
  a.seg_rows = in_place ? (int)(M / h->q) : 0;
  a.block_k = block_k_of(p);
  a.y_staged = 0;
  a.plan = nullptr;
  a.plan_stride = a.plan_rounds = a.plan_tag = 0;
  a.wait_limit = p.wait_limit;
  return cuda_status(launch_proj_tc(a, tc.tile_n, p.n_workers, st));
}

alg_status_t alg_proj_grad_last_status(alg_proj_grad_t h, void *stream, alg_status_t *status) {
  if (!h) return ALG_ERR_INVALID_ARG;
  return read_status(h->dx.d_status, stream, status);
}

static alg_status_t ffn_create(alg_ffn_t *out, int q, const int32_t *d_widths, const int32_t *f_widths,
                               alg_dtype_t dtype, alg_table_t table, const uint8_t *custom_keep,
                               alg_schedule_t schedule, bool gated) {
  if (!out) return ALG_ERR_INVALID_ARG;
  *out = nullptr;
  if (gated && dtype != ALG_BF16) return ALG_ERR_UNSUPPORTED_SHAPE;
  alg_ffn_s *f = new (std::nothrow) alg_ffn_s();
  if (!f) return ALG_ERR_INVALID_ARG;
  f->gated = gated;
  if (q > kMaxQ) {   // large-algebra handles are single projections
    delete f;
    return q > kBigMaxQ || q < 1 ? ALG_ERR_INVALID_ARG : ALG_ERR_UNSUPPORTED_SHAPE;
  }
  // (allow_big: with explicit types an FFN whose law and widths fit may run its projections on the large-algebra kernel)
  alg_status_t s = init_proj(f->up, q, d_widths, f_widths, dtype, table, custom_keep, schedule, nullptr, gated, true);
  if (s == ALG_OK) s = init_proj(f->down, q, f_widths, d_widths, dtype, table, custom_keep, schedule, f->up.d_status, false, true);
  if (s == ALG_OK && (f->up.big.only || f->down.big.only)) s = ALG_ERR_UNSUPPORTED_SHAPE;   // (interval schedule on the large-algebra path)
  if (s != ALG_OK) {
    free_proj(f->down);
    free_proj(f->up);
    delete f;
    return s;
  }
  f->D = f->up.K;
  f->F = f->up.N;
  if (dtype == ALG_BF16 && !gated && schedule != ALG_SCHED_INTERVAL &&
      ffn_decode_plan(q, f->up.s, f->down.s, f->D, f->F, f->up.num_sms, &f->fd)) {
    f->fd_ok = cudaMalloc(&f->d_counters, 2 * sizeof(unsigned int)) == cudaSuccess &&
               cudaMemset(f->d_counters, 0, 2 * sizeof(unsigned int)) == cudaSuccess;
  }
  if (dtype == ALG_BF16 && schedule != ALG_SCHED_INTERVAL && f->up.big.eligible && f->down.big.eligible &&
      row_decode_fits(q, f->D, f->F)) {
    // (the two one-launch decode kernels share the exchange counters: both leave them zero)
    f->rd_ok = f->d_counters != nullptr || (cudaMalloc(&f->d_counters, 2 * sizeof(unsigned int)) == cudaSuccess &&
                                            cudaMemset(f->d_counters, 0, 2 * sizeof(unsigned int)) == cudaSuccess);
  }
  *out = f;
  return ALG_OK;
}

alg_status_t alg_ffn_create(alg_ffn_t *out, int q, const int32_t *d_widths, const int32_t *f_widths,
                            alg_dtype_t dtype, alg_table_t table, const uint8_t *custom_keep,
                            alg_schedule_t schedule) {
  return ffn_create(out, q, d_widths, f_widths, dtype, table, custom_keep, schedule, false);
}

alg_status_t alg_ffn_gated_create(alg_ffn_t *out, int q, const int32_t *d_widths, const int32_t *f_widths,
                                  alg_dtype_t dtype, alg_table_t table, const uint8_t *custom_keep,
                                  alg_schedule_t schedule) {
  return ffn_create(out, q, d_widths, f_widths, dtype, table, custom_keep, schedule, true);
}

alg_status_t alg_ffn_gated_forward(alg_ffn_t h, const void *X, const int32_t *types, int64_t M, const void *W_gate_up,
                                   const void *W_down, void *Y, alg_dtype_t y_dtype, void *workspace,
                                   size_t workspace_bytes, void *stream) {
  if (!h || !h->gated) return ALG_ERR_INVALID_ARG;
  return alg_ffn_forward(h, X, types, M, W_gate_up, nullptr, W_down, nullptr, ALG_ACT_NONE, Y, y_dtype, workspace,
                         workspace_bytes, stream);
}

alg_status_t alg_ffn_destroy(alg_ffn_t h) {
  if (!h) return ALG_ERR_INVALID_ARG;
  for (int e = 0; e < 5; ++e)
    if (h->ev[e]) cudaEventDestroy(h->ev[e]);
  if (h->d_counters) cudaFree(h->d_counters);
  free_proj(h->down);
  free_proj(h->up);
  delete h;
  return ALG_OK;
}

alg_status_t alg_ffn_workspace_bytes(alg_ffn_t h, int64_t max_M, size_t *bytes) {
  if (!h || !bytes || max_M < 0 || max_M > (1 << 30)) return ALG_ERR_INVALID_ARG;
  *bytes = layout(h->up, &h->down, max_M).total;
  return ALG_OK;
}

alg_status_t alg_ffn_forward(alg_ffn_t h, const void *X, const int32_t *types, int64_t M, const void *W_up,
                             const void *b_up, const void *W_down, const void *b_down, alg_act_t act, void *Y,
                             alg_dtype_t y_dtype, void *workspace, size_t workspace_bytes, void *stream) {
  if (!h || M < 0 || M > (1 << 30)) return ALG_ERR_INVALID_ARG;
  if (M == 0) return ALG_OK;
  if (!X || !W_up || !W_down || !Y || !workspace) return ALG_ERR_INVALID_ARG;
  if (h->up.sched == ALG_SCHED_EXPLICIT && !types) return ALG_ERR_INVALID_ARG;
  if (y_dtype != ALG_F32 && y_dtype != ALG_BF16) return ALG_ERR_INVALID_ARG;
  if ((int)act < 0 || (int)act > 2) return ALG_ERR_INVALID_ARG;
  if (((uintptr_t)workspace & 255u) != 0) return ALG_ERR_INVALID_ARG;
  const int eb = elem_bytes(h->up.dtype);
  if (!aligned16(X) || !aligned16(W_up) || !aligned16(W_down) || !aligned16(Y)) return ALG_ERR_INVALID_ARG;
  if ((h->D * eb) % 16 || (h->F * eb) % 16 || (h->D * elem_bytes(y_dtype)) % 16) return ALG_ERR_INVALID_ARG;
  const WsLayout L = layout(h->up, &h->down, M);
  if (workspace_bytes < L.total) return ALG_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = (cudaStream_t)stream;
  char *ws = (char *)workspace;
  if (h->fd_ok && (h->up.opt_small_m == 1 || h->up.opt_small_m == 2 || (h->up.opt_small_m == 3 && !h->rd_ok)) && M <= kFfnDecodeMaxM && !h->timing) {
    // decode step in one launch: both projections, H exchanged through L2 inside the kernel
    const alg_proj_s &u = h->up;
    FfnDecodeArgs d = {};
    d.X = X;
    d.types = u.sched == ALG_SCHED_CYCLIC ? nullptr : types;
    d.M = (int)M;
    d.W_up = W_up, d.W_down = W_down;
    d.b_up = b_up, d.b_down = b_down;
    d.act = (int)act;
    d.H = ws + L.h;
    d.Y = Y;
    d.y_bf16 = y_dtype == ALG_BF16;
    d.D = h->D, d.F = h->F, d.q = u.q;
    d.counters = h->d_counters;
    d.status = u.d_status;
    d.wait_limit = u.wait_limit;
    d.extra_expect_bytes = u.test_extra_expect;
    d.tab_up = u.d_tab, d.tab_dn = h->down.d_tab;
    d.small_q = u.q <= kDecodeParamQ;
    if (d.small_q) {
      for (int e = 0; e <= u.q; ++e) d.so_d[e] = u.tab.so[e], d.so_f[e] = h->down.tab.so[e];
      for (int e = 0; e < u.q * u.q; ++e) d.keep[e] = u.tab.keep[e];
    }
    return cuda_status(launch_ffn_decode(d, h->fd, st));
  }
  if (h->rd_ok && (h->up.opt_small_m == 1 || h->up.opt_small_m == 3) &&
      M <= (h->up.opt_small_m == 3 ? kRowDecodeMaxM : row_decode_rows_ffn(h->up.q, h->D, h->F, h->gated)) && !h->timing && (!b_up || aligned16(b_up)) && (!b_down || aligned16(b_down))) {
    // decode step of one row in one launch
    if (h->gated && (b_up || b_down || act != ALG_ACT_NONE)) return ALG_ERR_INVALID_ARG;   // bias-free, silu(gate) * up
    RowDecodeArgs d = {};
    d.mode = h->gated ? 0 : 1;
    d.M = (int)M;
    d.X = X, d.ldx = h->D;
    d.types = h->up.sched == ALG_SCHED_CYCLIC ? nullptr : types;
    d.W1 = W_up, d.ldw1 = h->gated ? 2 * (int64_t)h->F : h->F;
    d.W2 = W_down, d.ldw2 = h->D;
    d.b1 = b_up, d.b2 = b_down;
    d.act = (int)act;
    d.H = ws + L.h;
    d.Y = Y, d.ldy = h->D;
    d.y_bf16 = y_dtype == ALG_BF16;
    d.D = h->D, d.F = h->F, d.q = h->up.q;
    d.counters = h->d_counters;
    d.status = h->up.d_status;
    d.wait_limit = h->up.wait_limit;
    d.extra_arrivals = h->up.test_extra_expect ? 1 : 0;
    return cuda_status(launch_row_decode(d, h->up.num_sms, st));
  }
  if (use_decode(h->up, M) && use_decode(h->down, M)) {
    // decode shapes: no bucketing, H stays in the original row order
    void *Hd = ws + L.h;
    alg_status_t sd = run_decode(h->up, X, h->D, types, M, W_up, h->F, b_up, act, Hd, h->F, ALG_BF16, st);
    if (sd != ALG_OK) return sd;
    return run_decode(h->down, Hd, h->F, types, M, W_down, h->D, b_down, ALG_ACT_NONE, Y, h->D, y_dtype, st);
  }

  BucketArgs b;
  b.types = h->up.sched == ALG_SCHED_CYCLIC ? nullptr : types;
  b.M = (int)M;
  b.q = h->up.q;
  b.chunk_rows = bucket_chunk_rows(M);
  b.hdr = (WsHeader *)(ws + L.hdr);
  b.chunk_counts = (int *)(ws + L.chunks);
  b.perm = (int *)(ws + L.perm);
  b.status = h->up.d_status;
  b.sync = (unsigned int *)(h->up.d_status + 2);
  b.wait_limit = h->up.wait_limit;
  b.Y = Y;
  b.ldy = h->D;
  b.N = h->D;
  b.y_elem_bytes = elem_bytes(y_dtype);
  const bool tm = h->timing;
  if (tm) cudaEventRecord(h->ev[0], st);
  int run_rows = 0;
  int64_t run_period = 0;
  if (h->up.sched == ALG_SCHED_INTERVAL && !interval_runs(h->up, M, &run_rows, &run_period)) return ALG_ERR_INVALID_ARG;
  const bool cyc = run_rows > 0 ||
                   (h->up.sched == ALG_SCHED_CYCLIC && M % h->up.q == 0 &&
                    ((use_tc(h->up) && use_tc(h->down)) || (use_big_equal(h->up, M) && use_big_equal(h->down, M))));
  if (!cyc && launch_bucket(b, st) != cudaSuccess) return ALG_ERR_CUDA;
  if (tm) cudaEventRecord(h->ev[1], st);
  void *H = ws + L.h;
  if (h->gated && (b_up || b_down || act != ALG_ACT_NONE)) return ALG_ERR_INVALID_ARG;   // bias-free, silu(gate) * up
  alg_status_t s = run_proj(h->up, L, ws, X, h->D, false, W_up, h->gated ? 2 * (int64_t)h->F : h->F, b_up, act, H, h->F,
                            h->up.dtype, true, M, st, tm ? h->ev[2] : nullptr, cyc, run_rows, run_period);
  if (s != ALG_OK) return s;
  if (tm) cudaEventRecord(h->ev[3], st);
  s = run_proj(h->down, L, ws, H, h->F, true, W_down, h->D, b_down, ALG_ACT_NONE, Y, h->D, y_dtype, false, M, st,
               nullptr, cyc, run_rows, run_period);
  if (tm) cudaEventRecord(h->ev[4], st);
  return s;
}

alg_status_t alg_ffn_set_timing(alg_ffn_t h, int enable) {
  if (!h) return ALG_ERR_INVALID_ARG;
  if (enable && !h->ev[0]) {
    for (int e = 0; e < 5; ++e)
      if (cudaEventCreate(&h->ev[e]) != cudaSuccess) return ALG_ERR_CUDA;
  }
  h->timing = enable != 0;
  return ALG_OK;
}

alg_status_t alg_ffn_get_timing(alg_ffn_t h, float *ms) {
  if (!h || !ms || !h->ev[0]) return ALG_ERR_INVALID_ARG;
  if (cudaEventSynchronize(h->ev[4]) != cudaSuccess) return ALG_ERR_CUDA;
  for (int e = 0; e < 4; ++e)
    if (cudaEventElapsedTime(&ms[e], h->ev[e], h->ev[e + 1]) != cudaSuccess) return ALG_ERR_CUDA;
  return ALG_OK;
}

alg_status_t alg_ffn_host_workspace_bytes(alg_ffn_t h, int64_t max_M, alg_dtype_t y_dtype, size_t *bytes) {
  if (!h || !bytes || max_M < 0 || max_M > (1 << 30)) return ALG_ERR_INVALID_ARG;
  if (y_dtype != ALG_F32 && y_dtype != ALG_BF16) return ALG_ERR_INVALID_ARG;
  size_t dev = layout(h->up, &h->down, max_M).total;
  size_t x = align_up((size_t)max_M * h->D * elem_bytes(h->up.dtype));
  size_t t = align_up((size_t)max_M * sizeof(int32_t));
  size_t y = align_up((size_t)max_M * h->D * elem_bytes(y_dtype));
  *bytes = align_up(dev) + x + t + y;
  return ALG_OK;
}

alg_status_t alg_ffn_forward_host(alg_ffn_t h, const void *X_host, const int32_t *types_host, int64_t M,
                                  const void *W_up, const void *b_up, const void *W_down, const void *b_down,
                                  alg_act_t act, void *Y_host, alg_dtype_t y_dtype, void *workspace,
                                  size_t workspace_bytes, void *stream) {
  if (!h || M < 0 || M > (1 << 30)) return ALG_ERR_INVALID_ARG;
  if (M == 0) return ALG_OK;
  if (!X_host || !Y_host || !workspace) return ALG_ERR_INVALID_ARG;
  if (h->up.sched == ALG_SCHED_EXPLICIT && !types_host) return ALG_ERR_INVALID_ARG;
  if (y_dtype != ALG_F32 && y_dtype != ALG_BF16) return ALG_ERR_INVALID_ARG;
  size_t need = 0;
  alg_status_t s = alg_ffn_host_workspace_bytes(h, M, y_dtype, &need);
  if (s != ALG_OK) return s;
  if (workspace_bytes < need) return ALG_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = (cudaStream_t)stream;
  char *ws = (char *)workspace;
  const size_t dev = align_up(layout(h->up, &h->down, M).total);
  const size_t xb = (size_t)M * h->D * elem_bytes(h->up.dtype);
  const size_t tb = (size_t)M * sizeof(int32_t);
  const size_t yb = (size_t)M * h->D * elem_bytes(y_dtype);
  char *dX = ws + dev;
  char *dT = dX + align_up(xb);
  char *dY = dT + align_up(tb);
  if (cudaMemcpyAsync(dX, X_host, xb, cudaMemcpyHostToDevice, st) != cudaSuccess) return ALG_ERR_CUDA;
  if (types_host && cudaMemcpyAsync(dT, types_host, tb, cudaMemcpyHostToDevice, st) != cudaSuccess) return ALG_ERR_CUDA;
  s = alg_ffn_forward(h, dX, types_host ? (const int32_t *)dT : nullptr, M, W_up, b_up, W_down, b_down, act, dY,
                      y_dtype, ws, dev, st);
  if (s != ALG_OK) return s;
  if (cudaMemcpyAsync(Y_host, dY, yb, cudaMemcpyDeviceToHost, st) != cudaSuccess) return ALG_ERR_CUDA;
  return ALG_OK;
}

alg_status_t alg_ffn_macs(alg_ffn_t h, const int64_t *rows_per_type, int64_t *macs) {
  if (!h || !macs) return ALG_ERR_INVALID_ARG;
  int64_t a = 0, b = 0;
  alg_status_t s = alg_proj_macs(&h->up, rows_per_type, &a);
  if (s != ALG_OK) return s;
  s = alg_proj_macs(&h->down, rows_per_type, &b);
  if (s != ALG_OK) return s;
  *macs = (h->gated ? 2 * a : a) + b;   // gate and up are two D x F projections
  return ALG_OK;
}

alg_status_t alg_ffn_last_status(alg_ffn_t h, void *stream, alg_status_t *status) {
  if (!h) return ALG_ERR_INVALID_ARG;
  alg_status_t s = read_status(h->up.d_status, stream, status);
  // a launch that gave up may have left the exchange counters of the one-launch decode step half way
  if (s == ALG_OK && *status != ALG_OK && h->d_counters)
    s = cuda_status(cudaMemset(h->d_counters, 0, 2 * sizeof(unsigned int)));
  return s;
}

const char *alg_status_string(alg_status_t s) {
  switch (s) {
    case ALG_OK: return "ok";
    case ALG_ERR_INVALID_ARG: return "invalid argument";
    case ALG_ERR_UNSUPPORTED_SHAPE: return "unsupported shape or device";
    case ALG_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case ALG_ERR_CUDA: return "CUDA call failed";
    case ALG_ERR_BAD_TYPE: return "row type outside [0, q)";
    case ALG_ERR_DEVICE_TIMEOUT: return "bounded device wait expired";
  }
  return "unknown status";
}

}  // extern "C"

namespace algproj {
int handle_device(alg_proj_t h) { return h ? h->device : -1; }
}  // namespace algproj

extern "C" {

int64_t alg_launch_count(void) { return algproj::g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
