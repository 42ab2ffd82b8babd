// C-ABI entry points: handle creation (interaction-table expansion, kernel selection), argument
// validation, workspace layout and the launch sequence of one forward pass.
#include <algorithm>
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "common.cuh"

using namespace algproj;

namespace algproj {
static std::atomic<int64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }
}  // namespace algproj

struct alg_proj_s {
  int q = 0;
  int s[kMaxQ] = {0}, r[kMaxQ] = {0};
  int K = 0, N = 0;
  alg_dtype_t dtype = ALG_F32;
  alg_schedule_t sched = ALG_SCHED_EXPLICIT;
  DevTable tab;             // host copy
  DevTable *d_tab = nullptr;
  int *d_status = nullptr;  // owned unless `shared_status`
  bool shared_status = false;
  bool tc_ok = false;
  bool pair_kernel = false; // cta_group::2 kernel (256-row tiles)
  int tile_n = 0;           // tensor-core tile width of the one-CTA kernel
  int device = 0;
  int num_sms = 148;
  int n_workers = 1;        // persistent CTAs (or CTA pairs) of the tensor-core kernel
  bool decode_ok = false;   // the small-M weight-streaming kernel covers this shape
  DecodePlan decode = {};
  // cyclic schedule: per-worker tile sequences for the last M seen, planned on the host
  TileRec *d_plan = nullptr, *h_plan = nullptr;  // n_workers x plan_stride records (device / pinned host)
  int plan_stride = 0, plan_rounds = 0;
  int64_t plan_M = -1;
  int plan_alternate = 0;
};

struct alg_ffn_s {
  alg_proj_s up, down;
  int D = 0, F = 0;
  bool timing = false;       // record events between the kernels of each forward call
  cudaEvent_t ev[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};
  // one-kernel FFN (cyclic schedule, bf16, q <= 8): host plan for the last M seen
  bool fused_ok = false;
  TileRec *d_fplan = nullptr, *h_fplan = nullptr;
  TileExt *d_fext = nullptr, *h_fext = nullptr;
  unsigned long long *d_counters = nullptr;
  int fused_workers = 0, fused_rounds = 0, fused_blocks = 0, fused_target = 0;
  int64_t fused_M = -1;
};

namespace {

long long *g_trace = nullptr;  // debug timeline buffer of the tensor-core kernel
int g_trace_cap = 0;

size_t align_up(size_t v, size_t a = 256) { return (v + a - 1) / a * a; }

bool use_tc(const alg_proj_s &p) { return p.dtype == ALG_BF16 && p.tc_ok; }
int tile_m_of(const alg_proj_s &p) { return !use_tc(p) ? 64 : p.pair_kernel ? kTc2TileM : kTcTileM; }
int tile_n_of(const alg_proj_s &p) { return !use_tc(p) ? 64 : p.pair_kernel ? kTc2TileN : p.tile_n; }
int elem_bytes(alg_dtype_t d) { return d == ALG_BF16 ? 2 : 4; }

alg_status_t init_proj(alg_proj_s &p, int q, const int32_t *in_w, const int32_t *out_w, alg_dtype_t dtype,
                       alg_table_t table, const uint8_t *custom, alg_schedule_t sched, int *shared_status) {
  if (q < 1 || q > kMaxQ || !in_w || !out_w) return ALG_ERR_INVALID_ARG;
  if (dtype != ALG_F32 && dtype != ALG_BF16) return ALG_ERR_INVALID_ARG;
  if (table != ALG_TABLE_QQ && table != ALG_TABLE_DENSE && table != ALG_TABLE_CUSTOM && table != ALG_TABLE_Q2POW)
    return ALG_ERR_INVALID_ARG;
  if (table == ALG_TABLE_Q2POW && (q & (q - 1)) != 0) return ALG_ERR_INVALID_ARG;  // q must be a power of two
  if (table == ALG_TABLE_CUSTOM && !custom) return ALG_ERR_INVALID_ARG;
  if (sched != ALG_SCHED_EXPLICIT && sched != ALG_SCHED_CYCLIC) return ALG_ERR_INVALID_ARG;
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
  if (const char *tn = std::getenv("ALGPROJ_TILE_N")) {  // experiment: force a tile width that divides every group
    const int v = atoi(tn);
    if ((v == 256 && all256) || (v == 192 && all192) || (v == 128 && all128)) p.tile_n = v;
  }
  // CTA-pair kernel whenever every output group splits into 256-wide tiles plus a 128-wide rest
  // (measured: it wins only when every tile has a long K loop; short loops favour the one-CTA kernel)
  int min_klen = 1 << 30;
  for (int pr = 0; pr < q * q; ++pr) {
    int len = 0;
    for (int k = 0; k < q; ++k)
      if ((p.tab.keep[pr] >> k) & 1u) len += p.s[k];
    min_klen = std::min(min_klen, len);
  }
  p.pair_kernel = p.tc_ok && all128 && min_klen >= 4096 && std::getenv("ALGPROJ_ONE_CTA") == nullptr;
  if (std::getenv("ALGPROJ_PAIR") != nullptr) p.pair_kernel = p.tc_ok && all128;

  // tile classes sorted by cost = K length x tile width, most expensive first (stable)
  {
    const int tn = tile_n_of(p);
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
    p.tab.n_classes = (int)order.size();
    for (size_t e = 0; e < order.size(); ++e) p.tab.cls[e] = order[e].rec;
    p.tab.n_pairs = q * q;
  }

  if (cudaGetDevice(&p.device) != cudaSuccess) return ALG_ERR_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, p.device) != cudaSuccess) return ALG_ERR_CUDA;
  p.num_sms = prop.multiProcessorCount;
  if (prop.major != 10) return ALG_ERR_UNSUPPORTED_SHAPE;  // sm_100a code only
  if (cudaMalloc(&p.d_tab, sizeof(DevTable)) != cudaSuccess) return ALG_ERR_CUDA;
  if (cudaMemcpy(p.d_tab, &p.tab, sizeof(DevTable), cudaMemcpyHostToDevice) != cudaSuccess) return ALG_ERR_CUDA;
  if (shared_status) {
    p.d_status = shared_status;
    p.shared_status = true;
  } else {
    if (cudaMalloc(&p.d_status, sizeof(int)) != cudaSuccess) return ALG_ERR_CUDA;
    if (cudaMemset(p.d_status, 0, sizeof(int)) != cudaSuccess) return ALG_ERR_CUDA;
  }
  if (use_tc(p) && tc_init() != cudaSuccess) return ALG_ERR_CUDA;
  if (use_tc(p)) {
    p.n_workers = p.pair_kernel ? tc2_max_pairs(p.num_sms) : std::min(p.num_sms, kMaxWorkers);
    if (p.n_workers < 1) return ALG_ERR_CUDA;
  }
  if (use_tc(p) && sched == ALG_SCHED_CYCLIC && std::getenv("ALGPROJ_NO_PLAN") == nullptr) {
    p.plan_stride = p.pair_kernel ? kTc2SeqCap : kTcSeqCap;
    const size_t bytes = (size_t)p.n_workers * p.plan_stride * sizeof(TileRec);
    if (cudaMalloc(&p.d_plan, bytes) != cudaSuccess) return ALG_ERR_CUDA;
    if (cudaMallocHost(&p.h_plan, bytes) != cudaSuccess) return ALG_ERR_CUDA;
  }
  if (dtype == ALG_BF16 && std::getenv("ALGPROJ_NO_DECODE") == nullptr) {
    p.decode_ok = decode_plan(q, p.s, p.K, p.N, p.num_sms, &p.decode);
    for (int g = 0; g < q && p.decode_ok; ++g)
      if (p.r[g] % p.decode.sn) p.decode_ok = false;
  }
  return ALG_OK;
}

void free_proj(alg_proj_s &p) {
  if (p.d_plan) cudaFree(p.d_plan);
  if (p.h_plan) cudaFreeHost(p.h_plan);
  p.d_plan = p.h_plan = nullptr;
  if (p.d_tab) cudaFree(p.d_tab);
  if (p.d_status && !p.shared_status) cudaFree(p.d_status);
  p.d_tab = nullptr;
  p.d_status = nullptr;
}

struct WsLayout {
  size_t hdr = 0, chunks = 0, perm = 0, xb = 0, h = 0, total = 0;
};

// `second`: the down projection of an FFN (nullptr for a single projection).
WsLayout layout(const alg_proj_s &first, const alg_proj_s *second, int64_t M) {
  WsLayout L;
  size_t off = 0;
  L.hdr = off;
  off = align_up(off + sizeof(WsHeader));
  L.chunks = off;
  off = align_up(off + (size_t)kMaxBucketChunks * (first.q + 1) * sizeof(int));
  L.perm = off;
  off = align_up(off + (size_t)M * sizeof(int));
  if (use_tc(first)) {
    L.xb = off;
    off = align_up(off + (size_t)M * first.K * 2, 1024);
  }
  if (second) {
    L.h = off;
    off = align_up(off + (size_t)M * first.N * elem_bytes(first.dtype), 1024);
  }
  L.total = off;
  return L;
}

alg_status_t cuda_status(cudaError_t e) { return e == cudaSuccess ? ALG_OK : ALG_ERR_CUDA; }

// Host twin of the in-kernel tile enumeration for the cyclic schedule (equal buckets of M/q rows):
// cost-sorted classes, m-tile major inside a class, boustrophedon assignment of tile indices to
// workers, optional alternation of expensive and cheap tiles inside a worker.  Fills p.h_plan and
// copies it to the device on `st`; returns false when the sequences do not fit the plan stride
// (the kernels then plan for themselves).
bool prepare_cyclic_plan(alg_proj_s &p, int64_t M, int alternate, cudaStream_t st) {
  if (!p.d_plan) return false;
  if (p.plan_M == M && p.plan_alternate == alternate) return p.plan_rounds > 0;
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(st, &cap) != cudaSuccess || cap != cudaStreamCaptureStatusNone) return false;
  const int q = p.q, nc = p.tab.n_classes, tile_m = tile_m_of(p), nw = p.n_workers, stride = p.plan_stride;
  const int bucket = (int)(M / q);
  const int m_tiles = (bucket + tile_m - 1) / tile_m;
  std::vector<long long> prefix(nc + 1, 0);
  for (int c = 0; c < nc; ++c) prefix[c + 1] = prefix[c] + (long long)m_tiles * p.tab.cls[c].n_tiles;
  const long long total = prefix[nc];
  const long long all_rounds = (total + nw - 1) / nw;
  p.plan_M = M;
  p.plan_alternate = alternate;
  p.plan_rounds = 0;
  if (all_rounds + 1 > stride) return false;
  std::vector<int> nkb(q * q, 0);
  for (int pr = 0; pr < q * q; ++pr)
    for (int k = 0; k < q; ++k)
      if ((p.tab.keep[pr] >> k) & 1u) nkb[pr] += p.s[k] / kTcBlockK;
  auto snake = [&](long long round, int w) { return round * nw + ((round & 1) ? (nw - 1 - w) : w); };
  const int rounds = (int)all_rounds + 1;
  for (int w = 0; w < nw; ++w) {
    const int valid = all_rounds == 0 ? 0 : (int)all_rounds - 1 + (snake(all_rounds - 1, w) < total ? 1 : 0);
    for (int pos = 0; pos < rounds; ++pos) {
      TileRec rec;
      rec.row0 = -1, rec.rows = 0, rec.pair = 0, rec.n0 = 0;
      if (pos < valid) {
        const int round = !alternate ? pos : (pos & 1) ? valid - 1 - (pos >> 1) : (pos >> 1);
        const long long idx = snake(round, w);
        int c = (int)(std::upper_bound(prefix.begin(), prefix.end(), idx) - prefix.begin()) - 1;
        const ClassRec &r = p.tab.cls[c];
        const int loc = (int)(idx - prefix[c]), ntl = (int)r.n_tiles, mt = loc / ntl, nt = loc - mt * ntl;
        rec.row0 = (int)r.i * bucket + mt * tile_m;
        rec.rows = std::min(tile_m, bucket - mt * tile_m) | (nkb[(int)r.i * q + (int)r.j] << 16);
        rec.pair = ((int)r.i * q + (int)r.j) | ((int)r.cols << 16);
        rec.n0 = r.col0 + nt * (int)r.cols;
      }
      p.h_plan[(size_t)w * stride + pos] = rec;
    }
  }
  // the pinned buffer is rewritten only when M changes: wait for the copy, so that no copy of an
  // older plan can still be reading it then
  if (cudaMemcpyAsync(p.d_plan, p.h_plan, (size_t)nw * stride * sizeof(TileRec), cudaMemcpyHostToDevice, st) !=
          cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess) {
    p.plan_M = -1;
    return false;
  }
  p.plan_rounds = rounds;
  return true;
}

bool aligned16(const void *p) { return ((uintptr_t)p & 15u) == 0; }

alg_status_t run_proj(alg_proj_s &p, const WsLayout &L, char *ws, const void *X, int64_t ldx,
                      bool x_bucketed, const void *W, int64_t ldw, const void *bias, alg_act_t act, void *Y,
                      int64_t ldy, alg_dtype_t y_dtype, bool y_bucketed, int64_t M, cudaStream_t st,
                      cudaEvent_t after_gather = nullptr, bool cyclic = false) {
  ProjArgs a;
  a.tab = p.d_tab;
  a.offsets = cyclic ? nullptr : ((const WsHeader *)(ws + L.hdr))->offsets;
  a.cyclic_rows = cyclic ? (int)(M / p.q) : 0;
  a.n_classes = p.tab.n_classes;
  a.st.valid = p.q <= kParamQ && p.tab.n_classes <= 2 * kParamQ * kParamQ;
  if (a.st.valid) {
    for (int e = 0; e <= p.q; ++e) a.st.so[e] = p.tab.so[e], a.st.ro[e] = p.tab.ro[e];
    for (int e = 0; e < p.q * p.q; ++e) a.st.keep[e] = p.tab.keep[e];
    for (int e = 0; e < p.tab.n_classes; ++e) a.st.cls[e] = p.tab.cls[e];
  }
  a.geom.tile_m = tile_m_of(p);
  a.geom.tile_m_log2 = a.geom.tile_m == 256 ? 8 : a.geom.tile_m == 128 ? 7 : 6;
  a.geom.alternate = std::getenv("ALGPROJ_ALTERNATE") ? atoi(std::getenv("ALGPROJ_ALTERNATE")) : 0;
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
  a.b_3d = 0;
  a.y_staged = 0;
  a.plan = nullptr;
  a.plan_stride = a.plan_rounds = 0;
  if (cyclic && prepare_cyclic_plan(p, M, a.geom.alternate, st)) {
    a.plan = p.d_plan;
    a.plan_stride = p.plan_stride;
    a.plan_rounds = p.plan_rounds;
  }
  a.dbg = std::getenv("ALGPROJ_DBG") ? atoi(std::getenv("ALGPROJ_DBG")) : 0;
  a.trace = g_trace;
  a.trace_cap = g_trace_cap;
  if (use_tc(p)) {
    if (x_bucketed || cyclic) {
      a.X = X;
      a.ldx = ldx;
    } else {
      cudaError_t e = launch_gather_rows(X, ldx, (const int *)(ws + L.perm), (int)M, p.K, 2, ws + L.xb, st);
      if (e != cudaSuccess) return ALG_ERR_CUDA;
      a.X = ws + L.xb;
      a.ldx = p.K;
    }
    if (after_gather) cudaEventRecord(after_gather, st);
    a.in_perm = nullptr;
    if (p.pair_kernel) return cuda_status(launch_proj_tc2(a, p.num_sms, st));
    return cuda_status(launch_proj_tc(a, p.tile_n, p.n_workers, st));
  }
  if (after_gather) cudaEventRecord(after_gather, st);
  a.X = X;
  a.ldx = ldx;
  a.in_perm = x_bucketed ? nullptr : (const int *)(ws + L.perm);
  return cuda_status(launch_proj_simt(a, p.dtype == ALG_BF16, st));
}

bool use_decode(const alg_proj_s &p, int64_t M) { return p.decode_ok && M <= kDecodeMaxM; }

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
  d.trace = g_trace;
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
  alg_status_t s = init_proj(*p, q, in_widths, out_widths, dtype, table, custom_keep, schedule, nullptr);
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
  if (ldx < h->K || ldw < h->N || ldy < h->N) return ALG_ERR_INVALID_ARG;
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
  if (use_decode(*h, M)) return run_decode(*h, X, ldx, types, M, W, ldw, bias, act, Y, ldy, y_dtype, st);

  BucketArgs b;
  b.types = h->sched == ALG_SCHED_CYCLIC ? nullptr : types;
  b.M = (int)M;
  b.q = h->q;
  b.chunk_rows = bucket_chunk_rows(M);
  b.hdr = (WsHeader *)(ws + L.hdr);
  b.chunk_counts = (int *)(ws + L.chunks);
  b.perm = (int *)(ws + L.perm);
  b.status = h->d_status;
  b.Y = Y;
  b.ldy = ldy;
  b.N = h->N;
  b.y_elem_bytes = elem_bytes(y_dtype);
  // cyclic schedule with equal buckets: no counting, no permutation, no gather
  const bool cyc = h->sched == ALG_SCHED_CYCLIC && use_tc(*h) && M % h->q == 0;
  if (!cyc && launch_bucket(b, st) != cudaSuccess) return ALG_ERR_CUDA;
  return run_proj(*h, L, ws, X, ldx, false, W, ldw, bias, act, Y, ldy, y_dtype, false, M, st, nullptr, cyc);
}

alg_status_t alg_proj_gemm_count(alg_proj_t h, int64_t *n) {
  if (!h || !n) return ALG_ERR_INVALID_ARG;
  int64_t c = 0;
  for (int pr = 0; pr < h->q * h->q; ++pr) c += __builtin_popcount(h->tab.keep[pr]);
  *n = c;
  return ALG_OK;
}

alg_status_t alg_proj_macs(alg_proj_t h, const int64_t *rows_per_type, int64_t *macs) {
  if (!h || !rows_per_type || !macs) return ALG_ERR_INVALID_ARG;
  int64_t total = 0;
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
  *path = use_decode(*h, M) ? ALG_PATH_DECODE : use_tc(*h) ? ALG_PATH_TCGEN05 : ALG_PATH_SIMT;
  return ALG_OK;
}

static alg_status_t read_status(int *d_status, void *stream, alg_status_t *status) {
  if (!status) return ALG_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  int v = 0;
  if (cudaStreamSynchronize(st) != cudaSuccess) return ALG_ERR_CUDA;
  if (cudaMemcpy(&v, d_status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return ALG_ERR_CUDA;
  if (v != 0 && cudaMemset(d_status, 0, sizeof(int)) != cudaSuccess) return ALG_ERR_CUDA;
  *status = (alg_status_t)v;
  return ALG_OK;
}

alg_status_t alg_proj_last_status(alg_proj_t h, void *stream, alg_status_t *status) {
  if (!h) return ALG_ERR_INVALID_ARG;
  return read_status(h->d_status, stream, status);
}

alg_status_t alg_ffn_create(alg_ffn_t *out, int q, const int32_t *d_widths, const int32_t *f_widths,
                            alg_dtype_t dtype, alg_table_t table, const uint8_t *custom_keep,
                            alg_schedule_t schedule) {
  if (!out) return ALG_ERR_INVALID_ARG;
  *out = nullptr;
  alg_ffn_s *f = new (std::nothrow) alg_ffn_s();
  if (!f) return ALG_ERR_INVALID_ARG;
  alg_status_t s = init_proj(f->up, q, d_widths, f_widths, dtype, table, custom_keep, schedule, nullptr);
  if (s == ALG_OK) s = init_proj(f->down, q, f_widths, d_widths, dtype, table, custom_keep, schedule, f->up.d_status);
  if (s != ALG_OK) {
    free_proj(f->down);
    free_proj(f->up);
    delete f;
    return s;
  }
  f->D = f->up.K;
  f->F = f->up.N;
  // one-kernel FFN: cyclic schedule, bf16 tensor path, tables by value (q <= 8), hidden groups in
  // 256-column tiles, output groups in 256-, 192- or 128-column tiles
  constexpr int kMaxFusedBlocks = 4096;
  bool fused = schedule == ALG_SCHED_CYCLIC && use_tc(f->up) && use_tc(f->down) && q <= kParamQ &&
               std::getenv("ALGPROJ_FUSED") != nullptr;
  for (int g = 0; g < q && fused; ++g) fused = f_widths[g] % 256 == 0 && (d_widths[g] % 128 == 0 || d_widths[g] % 192 == 0);
  if (fused) {
    f->fused_workers = std::min(f->up.num_sms, kMaxWorkers);
    const size_t n = (size_t)f->fused_workers * kFfnSeqCap;
    fused = cudaMalloc(&f->d_fplan, n * sizeof(TileRec)) == cudaSuccess &&
            cudaMallocHost(&f->h_fplan, n * sizeof(TileRec)) == cudaSuccess &&
            cudaMalloc(&f->d_fext, n * sizeof(TileExt)) == cudaSuccess &&
            cudaMallocHost(&f->h_fext, n * sizeof(TileExt)) == cudaSuccess &&
            cudaMalloc(&f->d_counters, (kMaxFusedBlocks + 1) * sizeof(unsigned long long)) == cudaSuccess &&
            cudaMemset(f->d_counters, 0, (kMaxFusedBlocks + 1) * sizeof(unsigned long long)) == cudaSuccess;
  }
  f->fused_ok = fused;
  *out = f;
  return ALG_OK;
}

namespace {

// Host plan of the one-kernel FFN for M rows (cyclic schedule: q equal buckets of M/q rows).
// Up tiles: row block (type i, m-tile) x hidden group j x 256-column tile; down tiles: the same row
// block x output group j x column tiles (192 wide when that divides the group and 256 does not,
// else 256 wide plus one of 128).  Built as a simulated timeline (costs in cycles from device
// timelines); a list that is valid in one timeline cannot deadlock: a wait cycle would need two
// down tiles that each start before the other.  Returns false when the plan does not fit (the
// caller then runs the two projections as two kernels).
bool prepare_fused_plan(alg_ffn_s &h, int64_t M, cudaStream_t st) {
  if (!h.fused_ok) return false;
  if (h.fused_M == M) return h.fused_rounds > 0;
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(st, &cap) != cudaSuccess || cap != cudaStreamCaptureStatusNone) return false;
  h.fused_M = M;
  h.fused_rounds = 0;
  const alg_proj_s &up = h.up, &dn = h.down;
  const int q = up.q, nw = h.fused_workers;
  const int bucket = (int)(M / q), m_tiles = (bucket + kTcTileM - 1) / kTcTileM, n_blocks = q * m_tiles;
  if (n_blocks * q > 4096) return false;
  auto nkb_of = [&](const alg_proj_s &p, int i, int j) {
    int n = 0;
    for (int k = 0; k < q; ++k)
      if ((p.tab.keep[i * q + j] >> k) & 1u) n += p.s[k] / kTcBlockK;
    return n;
  };
  struct Item { TileRec rec; TileExt ext; double cost; int block; int group; uint32_t mask; };
  auto make = [&](const alg_proj_s &p, int i, int mt, int j, int col0, int cols, bool down) {
    Item it;
    const int nkb = nkb_of(p, i, j);
    it.rec.row0 = i * bucket + mt * kTcTileM;
    it.rec.rows = std::min(kTcTileM, bucket - mt * kTcTileM) | (nkb << 16);
    it.rec.pair = (i * q + j) | (cols << 16);
    it.rec.n0 = col0;
    it.block = i * m_tiles + mt;
    it.group = j;
    it.mask = p.tab.keep[i * q + j];
    it.ext.dep = down ? it.block : -1;
    it.ext.sig = down ? -1 : it.block * q + j;   // an up tile completes part of hidden group j of its row block
    // cycles: a K block beside a running epilogue, the GELU epilogue as a floor, fixed hand-over
    it.cost = down ? nkb * (cols == 256 ? 509.0 : cols == 192 ? 467.0 : 460.0) + 2000.0
                   : std::max(nkb * 640.0, 5300.0) + 700.0;
    return it;
  };
  std::vector<Item> ups, downs;
  for (int mt = 0; mt < m_tiles; ++mt)
    for (int i = 0; i < q; ++i) {
      for (int j = 0; j < q; ++j)
        for (int t = 0; t < up.r[j] / 256; ++t) ups.push_back(make(up, i, mt, j, up.tab.ro[j] + t * 256, 256, false));
      for (int j = 0; j < q; ++j) {
        const int width = dn.r[j];
        if (width % 256 && width % 192 == 0) {
          for (int t = 0; t < width / 192; ++t) downs.push_back(make(dn, i, mt, j, dn.tab.ro[j] + t * 192, 192, true));
        } else {
          for (int t = 0; t < width / 256; ++t) downs.push_back(make(dn, i, mt, j, dn.tab.ro[j] + t * 256, 256, true));
          if (width % 256) downs.push_back(make(dn, i, mt, j, dn.tab.ro[j] + (width / 256) * 256, 128, true));
        }
      }
    }
  // 1. which worker runs how much: longest-processing-time over ALL tiles (the down tiles are the
  //    long ones and go first; the up tiles follow row block by row block as the fine filler)
  std::vector<double> load(nw, 0.0);
  std::vector<std::vector<Item>> my_ups(nw), my_downs(nw);
  auto least = [&]() { return (int)(std::min_element(load.begin(), load.end()) - load.begin()); };
  std::vector<int> order(downs.size());
  for (size_t e = 0; e < downs.size(); ++e) order[e] = (int)e;
  std::stable_sort(order.begin(), order.end(), [&](int x, int y) { return downs[x].cost > downs[y].cost; });
  for (int e : order) {
    const int w = least();
    load[w] += downs[e].cost;
    my_downs[w].push_back(downs[e]);
  }
  for (const Item &it : ups) {
    const int w = least();
    load[w] += it.cost;
    my_ups[w].push_back(it);
  }
  // 2. simulated timeline of the up tiles: every worker runs its own first, in row-block order
  std::vector<std::vector<Item>> seq(nw);
  std::vector<double> free_at(nw, 5000.0), part_done((size_t)n_blocks * q, 0.0);
  const double kHandOver = 6000.0;  // last epilogue of the part, signal, counter poll
  for (int w = 0; w < nw; ++w)
    for (const Item &it : my_ups[w]) {
      free_at[w] += it.cost;
      double &d = part_done[(size_t)it.block * q + it.group];
      d = std::max(d, free_at[w]);
      seq[w].push_back(it);
    }
  // earliest start of a down tile: its first kept hidden group must be complete, a later one by the
  // time the K loop reaches it
  auto ready_at = [&](const Item &it) {
    double start = 0.0, before = 0.0;
    for (int k = 0; k < q; ++k) {
      if (!((it.mask >> k) & 1u)) continue;
      start = std::max(start, part_done[(size_t)it.block * q + k] + kHandOver - before);
      before += (dn.s[k] / kTcBlockK) * 467.0;
    }
    return start;
  };
  std::vector<double> block_done(downs.size(), 0.0);   // per down tile: when it may start
  for (size_t e = 0; e < downs.size(); ++e) block_done[e] = ready_at(downs[e]) - kHandOver;
  // 3. which down tile exactly: step 1 fixed how many tiles of which length a worker runs; tiles
  //    of equal length are interchangeable.  Event-driven: whenever a worker becomes free it takes,
  //    among the remaining tiles of the length it is due to run (longest first), the one whose
  //    row block completed LAST among those already complete (best fit: early row blocks stay
  //    available for workers that become free early), else the one that completes first.
  {
    std::vector<char> taken(downs.size(), 0);
    std::vector<size_t> next_slot(nw, 0);
    for (int w = 0; w < nw; ++w)
      std::stable_sort(my_downs[w].begin(), my_downs[w].end(), [](const Item &x, const Item &y) { return x.cost > y.cost; });
    size_t left = downs.size();
    while (left > 0) {
      int w = -1;
      for (int v = 0; v < nw; ++v)
        if (next_slot[v] < my_downs[v].size() && (w < 0 || free_at[v] < free_at[w])) w = v;
      if (w < 0) break;
      const double want = my_downs[w][next_slot[w]].cost;
      int best = -1;
      for (size_t e = 0; e < downs.size(); ++e) {
        if (taken[e] || downs[e].cost != want) continue;
        if (best < 0) { best = (int)e; continue; }
        const double rb = block_done[best] + kHandOver, re = block_done[e] + kHandOver;
        const bool b_ok = rb <= free_at[w], e_ok = re <= free_at[w];
        if (e_ok && (!b_ok || re > rb)) best = (int)e;          // latest among the ready ones
        else if (!e_ok && !b_ok && re < rb) best = (int)e;      // nothing ready: the first to become ready
      }
      taken[best] = 1;
      --left;
      ++next_slot[w];
      free_at[w] = std::max(free_at[w], block_done[best] + kHandOver) + downs[best].cost;
      seq[w].push_back(downs[best]);
    }
  }
  size_t rounds = 0;
  for (int w = 0; w < nw; ++w) rounds = std::max(rounds, seq[w].size());
  rounds += 1;
  if ((int)rounds > kFfnSeqCap) return false;
  if (const char *dump = std::getenv("ALGPROJ_PLAN_DUMP")) {
    for (int w = 0; w < nw; w += (dump[0] == 'a' ? 1 : 20)) {
      fprintf(stderr, "worker %d (model end %.0f):", w, free_at[w]);
      for (const Item &it : seq[w])
        fprintf(stderr, " %c%d(k%d,c%d)", it.ext.dep >= 0 ? 'D' : 'U', it.block, it.rec.rows >> 16, it.rec.pair >> 16);
      fprintf(stderr, "\n");
    }
  }
  TileRec end;
  end.row0 = -1, end.rows = 0, end.pair = 0, end.n0 = 0;
  const TileExt none = {-1, -1};
  for (int w = 0; w < nw; ++w)
    for (size_t pos = 0; pos < (size_t)kFfnSeqCap; ++pos) {
      h.h_fplan[(size_t)w * kFfnSeqCap + pos] = pos < seq[w].size() ? seq[w][pos].rec : end;
      h.h_fext[(size_t)w * kFfnSeqCap + pos] = pos < seq[w].size() ? seq[w][pos].ext : none;
    }
  const size_t n = (size_t)nw * kFfnSeqCap;
  if (cudaMemcpyAsync(h.d_fplan, h.h_fplan, n * sizeof(TileRec), cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemcpyAsync(h.d_fext, h.h_fext, n * sizeof(TileExt), cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess) {
    h.fused_M = -1;
    return false;
  }
  h.fused_rounds = (int)rounds;
  h.fused_blocks = n_blocks * q;
  return true;
}

// Argument block of one projection as the fused kernel needs it (tables by value).
void fill_fused_proj(ProjArgs &a, const alg_proj_s &p, const void *X, int64_t ldx, const void *W, int64_t ldw,
                     const void *bias, alg_act_t act, void *Y, int64_t ldy, alg_dtype_t y_dtype, int64_t M,
                     int a_cyclic_rows, int out_cyclic_rows) {
  std::memset(&a, 0, sizeof(a));
  a.tab = p.d_tab;
  a.n_classes = p.tab.n_classes;
  a.st.valid = 1;
  for (int e = 0; e <= p.q; ++e) a.st.so[e] = p.tab.so[e], a.st.ro[e] = p.tab.ro[e];
  for (int e = 0; e < p.q * p.q; ++e) a.st.keep[e] = p.tab.keep[e];
  a.q = p.q;
  a.X = X, a.ldx = ldx, a.W = W, a.ldw = ldw, a.bias = bias, a.act = (int)act;
  a.Y = Y, a.ldy = ldy, a.y_bf16 = y_dtype == ALG_BF16;
  a.M = (int)M, a.K = p.K, a.N = p.N;
  a.status = p.d_status;
  a.a_cyclic_rows = a_cyclic_rows;
  a.out_cyclic_rows = out_cyclic_rows;
  a.cyclic_rows = (int)(M / p.q);
  a.dbg = std::getenv("ALGPROJ_DBG") ? atoi(std::getenv("ALGPROJ_DBG")) : 0;
  a.trace = g_trace;
  a.trace_cap = g_trace_cap;
}

}  // namespace

alg_status_t alg_ffn_destroy(alg_ffn_t h) {
  if (!h) return ALG_ERR_INVALID_ARG;
  for (int e = 0; e < 5; ++e)
    if (h->ev[e]) cudaEventDestroy(h->ev[e]);
  if (h->d_fplan) cudaFree(h->d_fplan);
  if (h->h_fplan) cudaFreeHost(h->h_fplan);
  if (h->d_fext) cudaFree(h->d_fext);
  if (h->h_fext) cudaFreeHost(h->h_fext);
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
  b.Y = Y;
  b.ldy = h->D;
  b.N = h->D;
  b.y_elem_bytes = elem_bytes(y_dtype);
  const bool tm = h->timing;
  if (tm) cudaEventRecord(h->ev[0], st);
  const bool cyc = h->up.sched == ALG_SCHED_CYCLIC && use_tc(h->up) && use_tc(h->down) && M % h->up.q == 0;
  if (cyc && !tm && aligned16(ws + L.h) && prepare_fused_plan(*h, M, st)) {
    // both projections in one persistent kernel
    FfnArgs fa;
    void *Hf = ws + L.h;
    const int rows = (int)(M / h->up.q);
    fill_fused_proj(fa.p[0], h->up, X, h->D, W_up, h->F, b_up, act, Hf, h->F, ALG_BF16, M, rows, 0);
    fill_fused_proj(fa.p[1], h->down, Hf, h->F, W_down, h->D, b_down, ALG_ACT_NONE, Y, h->D, y_dtype, M, 0, rows);
    fa.plan = h->d_fplan;
    fa.ext = h->d_fext;
    fa.plan_stride = kFfnSeqCap;
    fa.plan_rounds = h->fused_rounds;
    fa.counters = h->d_counters;
    fa.n_counters = h->fused_blocks;
    for (int g = 0; g < kParamQ; ++g) fa.target[g] = g < h->up.q ? h->up.r[g] / 256 : 0;
    return cuda_status(launch_ffn_tc(fa, h->fused_workers, st));
  }
  if (!cyc && launch_bucket(b, st) != cudaSuccess) return ALG_ERR_CUDA;
  if (tm) cudaEventRecord(h->ev[1], st);
  void *H = ws + L.h;
  alg_status_t s = run_proj(h->up, L, ws, X, h->D, false, W_up, h->F, b_up, act, H, h->F, h->up.dtype, true, M, st,
                            tm ? h->ev[2] : nullptr, cyc);
  if (s != ALG_OK) return s;
  if (tm) cudaEventRecord(h->ev[3], st);
  s = run_proj(h->down, L, ws, H, h->F, true, W_down, h->D, b_down, ALG_ACT_NONE, Y, h->D, y_dtype, false, M, st,
               nullptr, cyc);
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
  *macs = a + b;
  return ALG_OK;
}

alg_status_t alg_ffn_last_status(alg_ffn_t h, void *stream, alg_status_t *status) {
  if (!h) return ALG_ERR_INVALID_ARG;
  return read_status(h->up.d_status, stream, status);
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

// Internal debug hook (not part of the public header): device buffer of 8*3*cap int64 slots that
// the first eight CTAs of the tensor-core kernel fill with (clock64 << 8 | tag) records.
void alg_debug_set_trace(void *device_buffer, int cap) {
  g_trace = (long long *)device_buffer;
  g_trace_cap = cap;
}

int64_t alg_launch_count(void) { return algproj::g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
