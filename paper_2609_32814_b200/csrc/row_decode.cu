// Decode step of ONE row (M = 1) under the complete-graph law with q equal groups, in ONE launch: a projection
// y = act(x *_q W + b), the FFN  y = act(x *_q W_up + b_up) *_q W_down + b_down, or the gated FFN
// y = (silu(x * W_gate) .* (x * W_up)) * W_down  (the M = 1 rows of the paper's kernel tables, appendix "Kernel
// Benchmark Details").
//
// A row of type i needs, for the output group j, the block W_ij of its row panel and the diagonal block W_jj
// (Eqs. typed-diag / typed-off): 2 s of the q s weight rows above every output column.  The step is a pair of
// matrix-vector products bound by memory LATENCY, so it runs on plain FMAs and is organised around the dependent
// round trips.  A warp owns a piece of 8 or 16 output columns (and, while there are more warps than pieces, a
// share of the weight rows); its lanes split the rows, every lane keeps up to 32 loads of 16 bytes in flight and
// reads the activations it needs straight from global memory -- no staging, one CTA barrier per phase at most.
// The first weight loads are issued before the launch's dependency resolves (weights do not depend on the previous
// kernel), those of W_down before the wait between the phases of an FFN.  Phase 1 of an FFN writes the hidden row h
// (bf16) to global memory; all CTAs meet at a counter (bounded wait); phase 2 is the same routine on h and W_down.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>

#include "common.cuh"
#include "trace.cuh"

namespace algproj {
ALG_TRACE_DEFINE(row_decode)
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kLoads = 32;   // 16-byte weight loads a lane keeps in flight
constexpr int kMaxPo = 8;     // a piece has at most 8 x 8 columns
constexpr int kPieceCols = 16;   // columns of a piece where the group width allows (32 and 64 measured the same or slower)

// One matrix-vector phase as the kernel sees it.
struct Phase {
  const __nv_bfloat16 *W;   // weight bank, `ldw` elements per row
  int64_t ldw;
  int s;                    // rows of one input group
  int group_w;              // columns of one output group
  float inv_group_w;
  int n_cols;               // output columns (GATED: the up columns sit n_cols further in the bank)
  int pc;                   // columns of a piece: 8, 16, 32 or 64
  int ks;                   // warps that share the rows of a piece: 1, 2, 4 or 8
};

__device__ __forceinline__ void unpack8(const uint4 &v, float *f) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    f[2 * e] = __uint_as_float(w[e] << 16);
    f[2 * e + 1] = __uint_as_float(w[e] & 0xFFFF0000u);
  }
}

// Where a lane stands in a piece: `sub` = which 8 columns, `lr` = which share of the rows.
struct Lane {
  int piece, part, sub, lr, rl, col, j;
  bool on;
};
// (ks and pc / 8 are powers of two: shifts, and the group of a column by a reciprocal -- the step is bound by latency,
// and a handful of integer divisions on the way to the first load are a few hundred cycles of it)
__device__ __forceinline__ Lane lane_of(const Phase &p, int unit) {
  Lane l;
  const int lane = threadIdx.x & 31, po = p.pc >> 3, po_sh = __ffs(po) - 1, ks_sh = __ffs(p.ks) - 1;
  l.piece = unit >> ks_sh, l.part = unit & (p.ks - 1);
  l.sub = lane & (po - 1), l.lr = lane >> po_sh, l.rl = 32 >> po_sh;
  l.col = l.piece * p.pc + 8 * l.sub;
  l.on = l.col < p.n_cols;
  int j = (int)(((float)l.col + 0.5f) * p.inv_group_w);   // exact below 2^22 columns up to one step, corrected here
  if (j * p.group_w > l.col) --j;
  if ((j + 1) * p.group_w <= l.col) ++j;
  l.j = l.on ? j : 0;
  return l;
}

// Unit (piece x share of its rows) of this warp in round rd.  The warps that share a piece sit in one CTA; the pieces
// go round-robin over the CTAs, so that every SM carries the same number of busy warps (768 pieces on 148 SMs: five or
// six warps each, not eight on 96 of them; measured equal to the blocked order -- the step is bound by the chain of
// round trips, not by any one SM).
__device__ __forceinline__ int unit_of(int rd, int ks) {
  const int warp = threadIdx.x >> 5, ks_sh = __ffs(ks) - 1, slot = warp >> ks_sh, part = warp & (ks - 1);
  const int piece = (rd * (kWarps >> ks_sh) + slot) * gridDim.x + blockIdx.x;
  return piece * ks + part;
}

// Loads of one chunk: rows r0 .. of both segments (the diagonal block of group j, then -- unless the row's own type is
// j -- its panel block), for the gate and, GATED, the up columns.  RC rows per segment and chunk.
template <bool GATED>
__device__ __forceinline__ void load_chunk(uint4 (&w)[kLoads], const Phase &p, const Lane &l, int type, int c0) {
  constexpr int RC = GATED ? kLoads / 4 : kLoads / 2;
  const int step = p.ks * l.rl, first = l.part * l.rl + l.lr;
  const int nr = ((p.s + step - 1) >> (__ffs(step) - 1)) - c0;   // rows of this chunk some lane has (the same in every lane)
#pragma unroll
  for (int sg = 0; sg < 2; ++sg) {
    const int g = sg == 0 ? l.j : type;
    const bool seg_on = l.on && (sg == 0 || type != l.j);
    const __nv_bfloat16 *base = p.W + (int64_t)g * p.s * p.ldw + l.col;
#pragma unroll
    for (int u = 0; u < RC; ++u) {
      if (u >= nr) break;
      const int kk = first + (c0 + u) * step;
      const bool ok = seg_on && kk < p.s;
      const __nv_bfloat16 *src = base + (int64_t)kk * p.ldw;
      w[(sg * RC + u) * (GATED ? 2 : 1)] = ok ? __ldg((const uint4 *)src) : make_uint4(0, 0, 0, 0);
      if (GATED) w[(sg * RC + u) * 2 + 1] = ok ? __ldg((const uint4 *)(src + p.n_cols)) : make_uint4(0, 0, 0, 0);
    }
  }
}

// acc[0..8) (gate or plain) and acc[8..16) (up) += x[kk] * w[kk][...] for one chunk.  x is read from global memory
// (FROM_L2: written by other CTAs of this launch).
template <bool GATED, bool FROM_L2>
__device__ __forceinline__ void fma_chunk(const uint4 (&w)[kLoads], const Phase &p, const Lane &l, int type, int c0,
                                          const __nv_bfloat16 *x, float (&acc)[16]) {
  constexpr int RC = GATED ? kLoads / 4 : kLoads / 2;
  const int step = p.ks * l.rl, first = l.part * l.rl + l.lr;
  const int nr = ((p.s + step - 1) >> (__ffs(step) - 1)) - c0;   // rows of this chunk some lane has (the same in every lane)
  float xv[2 * RC];
#pragma unroll
  for (int sg = 0; sg < 2; ++sg) {
    const int g = sg == 0 ? l.j : type;
    const bool seg_on = l.on && (sg == 0 || type != l.j);
#pragma unroll
    for (int u = 0; u < RC; ++u) {
      if (u >= nr) break;
      const int kk = first + (c0 + u) * step;
      unsigned short raw = 0;
      if (seg_on && kk < p.s) {
        const unsigned short *src = (const unsigned short *)(x + (int64_t)g * p.s + kk);
        raw = FROM_L2 ? __ldcg(src) : __ldg(src);
      }
      xv[sg * RC + u] = __uint_as_float((uint32_t)raw << 16);
    }
  }
#pragma unroll
  for (int e = 0; e < 2 * RC; ++e) {
    if ((e % RC) >= nr) continue;
    float f[8];
    unpack8(w[e * (GATED ? 2 : 1)], f);
#pragma unroll
    for (int cc = 0; cc < 8; ++cc) acc[cc] = fmaf(xv[e], f[cc], acc[cc]);
    if (GATED) {
      unpack8(w[e * 2 + 1], f);
#pragma unroll
      for (int cc = 0; cc < 8; ++cc) acc[8 + cc] = fmaf(xv[e], f[cc], acc[8 + cc]);
    }
  }
}

// One phase for the units of this warp.  `w` holds the first chunk of the first unit when have_first.  Results of a
// piece: lanes with lr == 0 of the warp with part == 0 call `emit(col, acc)`.
template <bool GATED, bool FROM_L2, typename Emit>
__device__ __forceinline__ void run_phase(const Phase &p, int type, const __nv_bfloat16 *x, uint4 (&w)[kLoads], bool have_first,
                                          int n_units, float *partial, Emit emit) {
  constexpr int RC = GATED ? kLoads / 4 : kLoads / 2;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int total_warps = gridDim.x * kWarps, po = p.pc >> 3;
  const int rounds = (n_units + total_warps - 1) / total_warps;
  for (int rd = 0; rd < rounds; ++rd) {
    const int unit = unit_of(rd, p.ks);
    Lane l = lane_of(p, unit);
    if (unit >= n_units) l.on = false;
    float acc[16];
#pragma unroll
    for (int cc = 0; cc < 16; ++cc) acc[cc] = 0.f;
    const int rows_per_lane = (p.s + p.ks * l.rl - 1) >> (__ffs(p.ks * l.rl) - 1);
    for (int c0 = 0; c0 < rows_per_lane; c0 += RC) {
      if (!(have_first && rd == 0 && c0 == 0)) load_chunk<GATED>(w, p, l, type, c0);
      fma_chunk<GATED, FROM_L2>(w, p, l, type, c0, x, acc);
    }
    // sum over the lanes that share the columns
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) {
      if (d >= po) {
#pragma unroll
        for (int cc = 0; cc < (GATED ? 16 : 8); ++cc) acc[cc] += __shfl_xor_sync(0xffffffffu, acc[cc], d);
      }
    }
    if (p.ks > 1) {   // the warps of a piece sit in one CTA
      if (lane < po) {
#pragma unroll
        for (int cc = 0; cc < 16; ++cc) partial[(warp * kMaxPo + lane) * 16 + cc] = acc[cc];
      }
      __syncthreads();
      if (l.part == 0 && lane < po) {
        for (int o = 1; o < p.ks; ++o)
#pragma unroll
          for (int cc = 0; cc < 16; ++cc) acc[cc] += partial[((warp + o) * kMaxPo + lane) * 16 + cc];
      }
      __syncthreads();
    }
    if (l.on && l.part == 0 && lane < po) emit(l.col, acc);
  }
}

__device__ __forceinline__ int read_type(const RowDecodeArgs &a) {
  const int t = a.types ? a.types[0] : 0;
  return t < 0 || t >= a.q ? -1 : t;
}

__device__ __forceinline__ float activate(float z, int act) {
  if (act == ALG_ACT_GELU_ERF) return 0.5f * z * (1.f + erff(z * 0.70710678118654752f));
  if (act == ALG_ACT_GELU_TANH) return 0.5f * z * (1.f + tanhf(0.79788456080286536f * (z + 0.044715f * z * z * z)));
  return z;
}

// eight results of a piece: + bias, activation, stored as bf16 or fp32
__device__ __forceinline__ void store8(const float (&acc)[16], int col, const void *bias, int act, void *out, bool out_bf16) {
  float v[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) v[e] = acc[e];
  if (bias) {
    float b[8];
    unpack8(__ldg((const uint4 *)((const __nv_bfloat16 *)bias + col)), b);
#pragma unroll
    for (int e = 0; e < 8; ++e) v[e] += b[e];
  }
  if (act != ALG_ACT_NONE) {
#pragma unroll
    for (int e = 0; e < 8; ++e) v[e] = activate(v[e], act);
  }
  if (out_bf16) {
    uint32_t o[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      __nv_bfloat162 pk = __floats2bfloat162_rn(v[2 * e], v[2 * e + 1]);
      o[e] = *(uint32_t *)&pk;
    }
    *(uint4 *)((__nv_bfloat16 *)out + col) = make_uint4(o[0], o[1], o[2], o[3]);
  } else {
    float4 *dst = (float4 *)((float *)out + col);
    dst[0] = make_float4(v[0], v[1], v[2], v[3]);
    dst[1] = make_float4(v[4], v[5], v[6], v[7]);
  }
}

// MODE 0: gated FFN, 1: FFN, 2: projection (W1 only)
template <int MODE>
__global__ void __launch_bounds__(kThreads, 1) row_decode_kernel(const RowDecodeArgs a) {
  constexpr bool GATED = MODE == 0, FFN = MODE != 2;
  __shared__ float partial[kWarps * kMaxPo * 16];
  __shared__ int s_abort;
  ALG_TRACE_VARS;
  if (threadIdx.x == 0) ALG_TRACE(0, 1);
  // phase 1 maps the D (projection: K) inputs to F (N) columns of W1; phase 2 maps F back to D through W2
  Phase p1, p2;
  p1.W = (const __nv_bfloat16 *)a.W1, p1.ldw = a.ldw1, p1.s = a.gs, p1.group_w = a.gr, p1.inv_group_w = a.inv_gr, p1.n_cols = a.F;
  p1.pc = a.pc1, p1.ks = a.ks1;
  p2.W = (const __nv_bfloat16 *)a.W2, p2.ldw = a.ldw2, p2.s = a.gr, p2.group_w = a.gs, p2.inv_group_w = a.inv_gs, p2.n_cols = a.D;
  p2.pc = a.pc2, p2.ks = a.ks2;
  const __nv_bfloat16 *X = (const __nv_bfloat16 *)a.X;
  __nv_bfloat16 *H = (__nv_bfloat16 *)a.H;
  const int warp = threadIdx.x >> 5;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (threadIdx.x == 0) s_abort = 0;

  // ---- before the dependency resolves: the row type as it stands now and the first W1 loads it asks for (the type
  // is read again after the wait) ----
  const int t_early = read_type(a);
  uint4 w[kLoads];
  {
    const int unit = unit_of(0, p1.ks);
    Lane l = lane_of(p1, unit);
    if (unit >= a.units1 || t_early < 0) l.on = false;
    load_chunk<GATED>(w, p1, l, max(t_early, 0), 0);
  }
  if (threadIdx.x == 0) ALG_TRACE(0, 2);
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (threadIdx.x == 0) ALG_TRACE(0, 3);
  const int type = read_type(a);   // (in flight while phase 1 runs on the early value)

  // ---- phase 1 on the type read early, again if the type has changed since.  Gated: h = silu(x * W_gate) .*
  // (x * W_up); FFN: h = act(x * W_up + b_up); projection: y = act(x * W + b) ----
  for (int pass = 0; pass < 2; ++pass) {
    const int t = pass == 0 ? t_early : type;
    if (pass == 1 && type == t_early) break;
    if (t < 0) continue;
    run_phase<GATED, false>(p1, t, X, w, pass == 0, a.units1, partial, [&](int col, const float (&acc)[16]) {
      if (GATED) {
        uint32_t o[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float g0 = acc[2 * e], g1 = acc[2 * e + 1];
          __nv_bfloat162 pk = __floats2bfloat162_rn(g0 / (1.f + __expf(-g0)) * acc[8 + 2 * e], g1 / (1.f + __expf(-g1)) * acc[8 + 2 * e + 1]);
          o[e] = *(uint32_t *)&pk;
        }
        *(uint4 *)(H + col) = make_uint4(o[0], o[1], o[2], o[3]);
      } else if (FFN) {
        store8(acc, col, a.b1, a.act, H, true);
      } else {
        store8(acc, col, a.b1, a.act, a.Y, a.y_bf16 != 0);
      }
    });
  }
  if (type < 0 && threadIdx.x == 0 && blockIdx.x == 0) atomicExch(a.status, (int)ALG_ERR_BAD_TYPE);   // y = 0
  if (threadIdx.x == 0) ALG_TRACE(0, 6);
  if (!FFN) {
    if (type < 0) {   // a row type outside [0, q): the row of Y is zero
      for (int c = blockIdx.x * kThreads + threadIdx.x; c < a.F; c += gridDim.x * kThreads) {
        if (a.y_bf16) ((__nv_bfloat16 *)a.Y)[c] = __float2bfloat16_rn(0.f);
        else ((float *)a.Y)[c] = 0.f;
      }
    }
    return;
  }

  // ---- the first W_down loads go out before the wait between the phases ----
  {
    const int unit = unit_of(0, p2.ks);
    Lane l = lane_of(p2, unit);
    if (unit >= a.units2 || type < 0) l.on = false;
    load_chunk<false>(w, p2, l, max(type, 0), 0);
  }

  // ---- all of h is written before any of it is read: arrive, then wait (bounded) for the other CTAs ----
  __syncthreads();
  if (threadIdx.x == 0) {
    ALG_TRACE(0, 8);
    __threadfence();
    atomicAdd(a.counters, 1u);
    const long long t0 = clock64();
    bool ok = false;
    while (!ok) {
      unsigned int seen;
      asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(a.counters) : "memory");
      ok = seen >= gridDim.x + (unsigned int)a.extra_arrivals;
      if (!ok && clock64() - t0 > a.wait_limit) break;
    }
    if (!ok) {
      s_abort = 1;
      atomicExch(a.status, (int)ALG_ERR_DEVICE_TIMEOUT);
    }
    __threadfence();
    ALG_TRACE(0, 9);
  }
  __syncthreads();

  // ---- phase 2: y = h * W_down (+ b_down) ----
  if (!s_abort) {
    if (type >= 0) {
      run_phase<false, true>(p2, type, H, w, true, a.units2, partial,
                             [&](int col, const float (&acc)[16]) { store8(acc, col, a.b2, ALG_ACT_NONE, a.Y, a.y_bf16 != 0); });
    } else {   // a row type outside [0, q): the row of Y is zero
      for (int c = blockIdx.x * kThreads + threadIdx.x; c < a.D; c += gridDim.x * kThreads) {
        if (a.y_bf16) ((__nv_bfloat16 *)a.Y)[c] = __float2bfloat16_rn(0.f);
        else ((float *)a.Y)[c] = 0.f;
      }
    }
  }
  // the last CTA past the wait clears the counters for the next launch
  if (threadIdx.x == 0) {
    ALG_TRACE(0, 12);
    const unsigned int left = atomicAdd(a.counters + 1, 1u);
    if (left == gridDim.x - 1) {
      a.counters[0] = 0;
      a.counters[1] = 0;
      __threadfence();
    }
  }
}

__device__ __forceinline__ int read_row_type(const RowDecodeArgs &a, int m) {
  const int t = a.types ? a.types[m] : m % a.q;
  return t < 0 || t >= a.q ? -1 : t;
}

// The same phase for several rows: unit = (row, piece, share of the piece's weight rows), rows outermost.  `w` holds
// the first chunk of the first unit when have_first, fetched for row type t_first; the other units read their row's
// type themselves.  Results of a piece: lanes with lr == 0 of the warp with part == 0 call `emit(row, col, acc)`.
// Barrier of the warps that share a piece (2, 4 or 8 of them: at most four groups per CTA).  The ids are literals so
// that the kernel reserves five hardware barriers, not all sixteen -- with sixteen a second CTA (the next launch's,
// which starts early to request its weights) could not become resident beside this one.
__device__ __forceinline__ void group_barrier(int id, int threads) {
  switch (id) {
    case 1: asm volatile("bar.sync 1, %0;" ::"r"(threads) : "memory"); break;
    case 2: asm volatile("bar.sync 2, %0;" ::"r"(threads) : "memory"); break;
    case 3: asm volatile("bar.sync 3, %0;" ::"r"(threads) : "memory"); break;
    default: asm volatile("bar.sync 4, %0;" ::"r"(threads) : "memory"); break;
  }
}

// A row whose type lies outside [0, q) reads nothing; with LAST (the phase that writes Y) its pieces are stored as zeros
// and the status word says so.
template <bool GATED, bool FROM_L2, bool LAST, typename Emit>
__device__ __forceinline__ void run_rows_phase(const RowDecodeArgs &a, const Phase &p, const __nv_bfloat16 *x, int64_t ldx,
                                          uint4 (&w)[kLoads], bool have_first, int t_first, int n_units, float *partial, Emit emit) {
  constexpr int RC = GATED ? kLoads / 4 : kLoads / 2;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int total_warps = gridDim.x * kWarps, po = p.pc >> 3;
  const int rounds = (n_units + total_warps - 1) / total_warps;
  const int per_row = a.M == 1 ? n_units : n_units / a.M;   // (one row: no division on the way to the first load)
  for (int rd = 0; rd < rounds; ++rd) {
    const int unit = unit_of(rd, p.ks);
    const int m = a.M == 1 ? 0 : min(unit / per_row, a.M - 1);
    const int real = read_row_type(a, m);   // (on its way while the first attempt below runs on the type read early)
    int type = have_first && rd == 0 ? t_first : real;
    const __nv_bfloat16 *xm = x + (int64_t)m * ldx;
    // the first unit runs on the type read before the launch's dependency resolved; if the type has changed since, the
    // warps of the piece (they share the row) do it again -- they meet at a barrier of their own, not the CTA's
    for (int attempt = 0; attempt < 2; ++attempt) {
      Lane l = lane_of(p, unit - m * per_row);
      if (unit >= n_units || type < 0) l.on = false;
      float acc[16];
#pragma unroll
      for (int cc = 0; cc < 16; ++cc) acc[cc] = 0.f;
      const int rows_per_lane = (p.s + p.ks * l.rl - 1) >> (__ffs(p.ks * l.rl) - 1);
      for (int c0 = 0; c0 < rows_per_lane; c0 += RC) {
        if (!(have_first && rd == 0 && attempt == 0 && c0 == 0)) load_chunk<GATED>(w, p, l, max(type, 0), c0);
        fma_chunk<GATED, FROM_L2>(w, p, l, max(type, 0), c0, xm, acc);
      }
      // sum over the lanes that share the columns
#pragma unroll
      for (int d = 16; d >= 1; d >>= 1) {
        if (d >= po) {
#pragma unroll
          for (int cc = 0; cc < (GATED ? 16 : 8); ++cc) acc[cc] += __shfl_xor_sync(0xffffffffu, acc[cc], d);
        }
      }
      if (p.ks > 1) {   // the warps of a piece sit side by side in one CTA
        const int bar_id = 1 + warp / p.ks, bar_threads = 32 * p.ks;
        if (lane < po) {
#pragma unroll
          for (int cc = 0; cc < 16; ++cc) partial[(warp * kMaxPo + lane) * 16 + cc] = acc[cc];
        }
        group_barrier(bar_id, bar_threads);
        if (l.part == 0 && lane < po) {
          for (int o = 1; o < p.ks; ++o)
#pragma unroll
            for (int cc = 0; cc < 16; ++cc) acc[cc] += partial[((warp + o) * kMaxPo + lane) * 16 + cc];
        }
        group_barrier(bar_id, bar_threads);
      }
      if (attempt == 0 && type != real) {
        type = real;
        continue;
      }
      if (l.on && l.part == 0 && lane < po) emit(m, l.col, acc);
      if (LAST && type < 0 && unit < n_units && l.part == 0 && lane < po && l.col < p.n_cols) {
        if (a.y_bf16) *(uint4 *)((__nv_bfloat16 *)a.Y + (int64_t)m * a.ldy + l.col) = make_uint4(0, 0, 0, 0);
        else ((float4 *)((float *)a.Y + (int64_t)m * a.ldy + l.col))[0] = ((float4 *)((float *)a.Y + (int64_t)m * a.ldy + l.col))[1] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (lane == 0) atomicExch(a.status, (int)ALG_ERR_BAD_TYPE);
      }
      break;
    }
  }
}

// Several rows (2 .. kRowDecodeMaxM): the row is the outermost dimension of the units; every warp reads the type of the
// rows it works on.  (A kernel of its own: the index arithmetic of the general form costs the one-row step 0.4-1 us.)
// MODE 0: gated FFN, 1: FFN, 2: projection (W1 only)
template <int MODE>
__global__ void __launch_bounds__(kThreads, 1) rows_decode_kernel(const RowDecodeArgs a) {
  constexpr bool GATED = MODE == 0, FFN = MODE != 2;
  __shared__ float partial[kWarps * kMaxPo * 16];
  __shared__ int s_abort;
  ALG_TRACE_VARS;
  if (threadIdx.x == 0) ALG_TRACE(0, 1);
  // phase 1 maps the D (projection: K) inputs to F (N) columns of W1; phase 2 maps F back to D through W2
  Phase p1, p2;
  p1.W = (const __nv_bfloat16 *)a.W1, p1.ldw = a.ldw1, p1.s = a.gs, p1.group_w = a.gr, p1.inv_group_w = a.inv_gr, p1.n_cols = a.F;
  p1.pc = a.pc1, p1.ks = a.ks1;
  p2.W = (const __nv_bfloat16 *)a.W2, p2.ldw = a.ldw2, p2.s = a.gr, p2.group_w = a.gs, p2.inv_group_w = a.inv_gs, p2.n_cols = a.D;
  p2.pc = a.pc2, p2.ks = a.ks2;
  const __nv_bfloat16 *X = (const __nv_bfloat16 *)a.X;
  __nv_bfloat16 *H = (__nv_bfloat16 *)a.H;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (threadIdx.x == 0) s_abort = 0;

  // ---- before the dependency resolves: the type of this warp's first row as it stands now and the first W1 loads it
  // asks for (the type is read again after the wait) ----
  const int per_row1 = a.M == 1 ? a.units1 : a.units1 / a.M;
  const int unit1 = unit_of(0, p1.ks), m1 = a.M == 1 ? 0 : min(unit1 / per_row1, a.M - 1);
  const int t_early = read_row_type(a, m1);
  uint4 w[kLoads];
  {
    Lane l = lane_of(p1, unit1 - m1 * per_row1);
    if (unit1 >= a.units1 || t_early < 0) l.on = false;
    load_chunk<GATED>(w, p1, l, max(t_early, 0), 0);
  }
  if (threadIdx.x == 0) ALG_TRACE(0, 2);
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (threadIdx.x == 0) ALG_TRACE(0, 3);

  // ---- phase 1 (its first unit on the type read early).  Gated: h = silu(x * W_gate) .* (x * W_up); FFN:
  // h = act(x * W_up + b_up); projection: y = act(x * W + b) ----
  {
    run_rows_phase<GATED, false, !FFN>(a, p1, X, a.ldx, w, true, t_early, a.units1, partial, [&](int m, int col, const float (&acc)[16]) {
      if (GATED) {
        uint32_t o[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float g0 = acc[2 * e], g1 = acc[2 * e + 1];
          __nv_bfloat162 pk = __floats2bfloat162_rn(g0 / (1.f + __expf(-g0)) * acc[8 + 2 * e], g1 / (1.f + __expf(-g1)) * acc[8 + 2 * e + 1]);
          o[e] = *(uint32_t *)&pk;
        }
        *(uint4 *)(H + (int64_t)m * a.F + col) = make_uint4(o[0], o[1], o[2], o[3]);
      } else if (FFN) {
        store8(acc, col, a.b1, a.act, H + (int64_t)m * a.F, true);
      } else {
        store8(acc, col, a.b1, a.act, a.y_bf16 ? (void *)((__nv_bfloat16 *)a.Y + (int64_t)m * a.ldy) : (void *)((float *)a.Y + (int64_t)m * a.ldy),
               a.y_bf16 != 0);
      }
    });
  }
  if (threadIdx.x == 0) ALG_TRACE(0, 6);

  if (FFN) {
    // ---- the first W_down loads go out before the wait between the phases ----
    const int per_row2 = a.M == 1 ? a.units2 : a.units2 / a.M;
    const int unit2 = unit_of(0, p2.ks), m2 = a.M == 1 ? 0 : min(unit2 / per_row2, a.M - 1);
    const int type2 = read_row_type(a, m2);
    {
      Lane l = lane_of(p2, unit2 - m2 * per_row2);
      if (unit2 >= a.units2 || type2 < 0) l.on = false;
      load_chunk<false>(w, p2, l, max(type2, 0), 0);
    }

    // ---- all of h is written before any of it is read: arrive, then wait (bounded) for the other CTAs ----
    __syncthreads();
    if (threadIdx.x == 0) {
      ALG_TRACE(0, 8);
      __threadfence();
      atomicAdd(a.counters, 1u);
      const long long t0 = clock64();
      bool ok = false;
      while (!ok) {
        unsigned int seen;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(a.counters) : "memory");
        ok = seen >= gridDim.x + (unsigned int)a.extra_arrivals;
        if (!ok && clock64() - t0 > a.wait_limit) break;
      }
      if (!ok) {
        s_abort = 1;
        atomicExch(a.status, (int)ALG_ERR_DEVICE_TIMEOUT);
      }
      __threadfence();
      ALG_TRACE(0, 9);
    }
    __syncthreads();

    // ---- phase 2: y = h * W_down (+ b_down) ----
    if (!s_abort) {
      run_rows_phase<false, true, true>(a, p2, H, a.F, w, true, type2, a.units2, partial, [&](int m, int col, const float (&acc)[16]) {
        store8(acc, col, a.b2, ALG_ACT_NONE,
               a.y_bf16 ? (void *)((__nv_bfloat16 *)a.Y + (int64_t)m * a.ldy) : (void *)((float *)a.Y + (int64_t)m * a.ldy), a.y_bf16 != 0);
      });
    }
    // the last CTA past the wait clears the counters for the next launch
    if (threadIdx.x == 0) {
      ALG_TRACE(0, 12);
      const unsigned int left = atomicAdd(a.counters + 1, 1u);
      if (left == gridDim.x - 1) {
        a.counters[0] = 0;
        a.counters[1] = 0;
        __threadfence();
      }
    }
  }

}

// warps per piece: as many (a power of two, at most the warps of a CTA) as the grid has warps for
int pick_ks(int pieces, int grid) {
  int ks = 1;
  while (ks < kWarps && pieces * ks * 2 <= grid * kWarps) ks *= 2;
  return ks;
}

template <int MODE>
cudaError_t launch_mode(const RowDecodeArgs &a, int grid, cudaStream_t st) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid, 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  cudaError_t e = a.M == 1 ? cudaLaunchKernelEx(&cfg, row_decode_kernel<MODE>, a) : cudaLaunchKernelEx(&cfg, rows_decode_kernel<MODE>, a);
  count_launch(1);
  return e;
}

}  // namespace

bool row_decode_fits(int q, int D, int F) {
  if (q < 1 || D % q || F % q) return false;
  return (D / q) % 8 == 0 && (F / q) % 8 == 0;
}

cudaError_t launch_row_decode(const RowDecodeArgs &in, int num_sms, cudaStream_t st) {
  RowDecodeArgs a = in;
  if (a.mode < 0 || a.mode > 2 || a.M < 1 || a.M > kRowDecodeMaxM || !row_decode_fits(a.q, a.D, a.F)) return cudaErrorInvalidValue;
  const int s = a.D / a.q, r = a.F / a.q;
  a.gs = s, a.gr = r, a.inv_gs = 1.f / (float)s, a.inv_gr = 1.f / (float)r;
  auto piece = [](int group_w) { return group_w % kPieceCols == 0 ? kPieceCols : group_w % 16 == 0 ? 16 : 8; };
  a.pc1 = piece(r);
  a.pc2 = piece(s);
  const int pieces1 = a.F / a.pc1, pieces2 = a.mode == 2 ? 0 : a.D / a.pc2;
  a.ks1 = pick_ks(pieces1 * a.M, num_sms);
  a.ks2 = pieces2 ? pick_ks(pieces2 * a.M, num_sms) : 1;
  a.units1 = a.M * pieces1 * a.ks1;
  a.units2 = a.M * pieces2 * a.ks2;
  // every CTA of an FFN must be resident for the wait between the phases: one CTA per SM at most
  const int grid = std::min(num_sms, std::max(a.units1 / a.ks1, a.units2 / a.ks2));   // at most one piece group per CTA and slot
  if (a.mode == 0) return launch_mode<0>(a, grid, st);
  if (a.mode == 1) return launch_mode<1>(a, grid, st);
  return launch_mode<2>(a, grid, st);
}

}  // namespace algproj
