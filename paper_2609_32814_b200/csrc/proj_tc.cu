// Grouped bf16 GEMM over the interaction table for sm_100a: TMA-fed shared-memory tiles,
// tcgen05.mma with the accumulator in tensor memory, persistent CTAs walking the tile
// enumeration (tile_map.cuh) in a static boustrophedon order.
//
// One output tile = 128 rows of one row type i  x  TILE_N columns of one output group j.  All
// kept products of that block (x_k W_kj for k in B(i,j); Eq. recursive-row-action -- for the
// Q_q law x_i W_ij + x_j W_jj, Eqs. typed-diag/off) are issued back to back into the SAME
// TMEM accumulator, so no partial sum ever reaches HBM (the fused forward kernel of Section
// "Kernels": every endpoint product of an output block is summed before the block is written).
//
// Operands: A = type-bucketed rows, K-contiguous (K-major), 128B-swizzled 128x64 tiles.
//           B = the canonical K x N bank, N-contiguous (MN-major), 64(k) x 64(n) swizzled boxes.
// Warp roles (352 threads): warp 0 = TMA producer of A (one lane), warp 10 = TMA producer of B,
// warp 1 = TMEM allocator + MMA issuer (one lane), warps 2..9 = epilogue (TMEM -> registers ->
// bias / activation -> row scatter to global; two warps per TMEM lane quadrant, each taking half
// the columns).  The
// accumulator is double buffered in TMEM so the epilogue of tile t overlaps the main loop of
// tile t+1.
//
// Every wait on an mbarrier is bounded: on expiry the CTA raises ALG_ERR_DEVICE_TIMEOUT in the
// handle's status word, all roles leave their loops, TMEM is released and the kernel returns.
#include <cudaTypedefs.h>

#include <cstring>

#include "tc_common.cuh"

namespace algproj {

using namespace tc;

ALG_TRACE_DEFINE(proj_tc)

namespace {

struct Ctl {
  uint64_t full[12];
  uint64_t empty[12];
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint32_t tmem_base;
  volatile int abort_flag;
  long long wait_limit;     // bound of every wait, in clock64 cycles
  // interaction table, copied once per CTA so no role waits on global metadata at a tile start
  int so[kMaxQ + 1];
  uint32_t keep[kMaxPairs];
  uint16_t nkb[kMaxPairs];  // K blocks per tile of a pair
};

// Bounded wait. Returns false when the CTA is aborting.
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
constexpr int kSeqCap = kTcSeqCap;  // precomputed tile records per CTA
#ifndef ALGPROJ_EPI_WARPS
#define ALGPROJ_EPI_WARPS 8
#endif
constexpr int kEpiWarps = ALGPROJ_EPI_WARPS;
constexpr int kProducerWarpB = 2 + kEpiWarps;   // second TMA producer, after the epilogue warps
constexpr int kThreads = 32 * (3 + kEpiWarps);

// TILE_M = 128: one accumulator of 128 rows x TILE_N columns per tile.
// TILE_M = 256: two accumulators (rows 0..127 and 128..255) side by side in tensor memory; every
// 64-deep B block is fetched once and used by two M = 128 MMAs, which cuts the operand bytes per
// multiply-accumulate by a quarter against a 128 x 192 tile -- the layout for projections with a
// long reduction and narrow output groups (TILE_N = 128 only, so that two tiles still fit the
// 512 columns and the epilogue of one tile overlaps the main loop of the next).
//
// BK = reduction depth of one pipeline stage, 64 or 32.  The bytes a CTA has in flight are what its
// operand fill rate hangs on (a freed stage is refilled one L2 round trip later); of S stages S - 1
// are in flight while one is consumed, so twice as many stages of half the depth keep 7/8 instead of
// 3/4 of the same shared memory busy.  BK = 32 rows of A are 64 bytes: 64-byte swizzle atoms there.
template <int TILE_N, int TILE_M, int BK>
struct Cfg {
  static constexpr int kHalves = TILE_M / 128;                  // accumulators (MMAs per K step) of a tile
  static constexpr int kAHalfBytes = 128 * BK * 2;              // 128 rows of A: 16 KB (BK = 64) or 8 KB
  static constexpr int kABytes = TILE_M * BK * 2;
  static constexpr int kBChunkBytes = BK * 64 * 2;              // one BK(k) x 64(n) box: 8 KB or 4 KB
  static constexpr int kBBytes = kBChunkBytes * (TILE_N / 64);
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kStages = (200 * 1024) / kStageBytes > 12 ? 12 : (200 * 1024) / kStageBytes;
  static constexpr uint32_t kSwzK = BK == 64 ? 2 : 4;            // descriptor swizzle mode of a K-major operand
  static constexpr uint32_t kSboK = 8 * BK * 2;                  // 8 rows of a K-major operand
  static constexpr int kAccStride = TILE_N * kHalves <= 128 ? 128 : 256;   // TMEM columns between the two tile buffers
  static constexpr int kTmemCols = 2 * kAccStride;
  static constexpr int kFixedSmemBytes = kStages * kStageBytes + (int)sizeof(Ctl) + kSeqCap * 16 + 16 + 1024;  // + tile map
  static constexpr int kStoreBufBytes = 32 * 64;                  // per epilogue warp: 32 rows x 32 bf16 columns
  // an epilogue warp takes 32 rows x kHalf columns: half of the columns of the one accumulator, or
  // all columns of one of the two accumulators
  static constexpr int kHalf = TILE_N * kHalves / (kEpiWarps / 4);
  // instruction descriptor: D=f32, A=B=bf16, A K-major, B MN-major, N, M=128
  static constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | (1u << 16) |
                                     ((uint32_t)(TILE_N >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
  static_assert(BK == 64 || BK == 32, "stage depth");
  static_assert(TILE_M == 128 || (TILE_M == 256 && TILE_N == 128), "256-row tiles are 128 columns wide");
  static_assert(kHalves == 1 || kEpiWarps == 8, "two accumulators need one epilogue warp group each");
};

// GATED (TILE_N = 256, TILE_M = 128 only): the SwiGLU up projection.  B is the merged bank
// [W_gate | W_up]; a stage holds the 128 gate columns of the tile followed by its 128 up columns, one
// N = 256 MMA fills both halves of the accumulator, and the epilogue writes silu(gate) * up -- 128
// output columns per tile, the hidden state is stored once and the two pre-activations never
// leave the chip (the merged gate/up kernel of the appendix "Kernel Benchmark Details").
constexpr int kGatherWarps = 6;   // AMODE 2: extra warps that only issue row gathers, after the B producer
constexpr int kGatherLanes = 32 / (2 + kGatherWarps);   // lanes of a warp that issue gathers
template <int TILE_N, int TILE_M, bool GATED, int BK, int AMODE>
__global__ void __launch_bounds__(AMODE == 2 ? kThreads + 32 * kGatherWarps : kThreads, 1)
proj_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const ProjArgs a) {
  using C = Cfg<TILE_N, TILE_M, BK>;
  static_assert(!GATED || (TILE_N == 256 && TILE_M == 128), "the gated kernel pairs two 128-column halves");
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  // optional staging buffers of the epilogue warps sit between the stages and the control block
  uint8_t *store_buf = smem + C::kStages * C::kStageBytes;
  Ctl *ctl = (Ctl *)(store_buf + (a.y_staged ? kEpiWarps * C::kStoreBufBytes : 0));
  TileRec *recs = (TileRec *)(ctl + 1);
  TileMap *tm = (TileMap *)(recs + kSeqCap);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const DevTable *__restrict__ tab = a.tab;
  const int q = a.q;
  ALG_TRACE_VARS;
  ALG_TRACE_CTA(0, a.act ? 0 : 1);

  if (threadIdx.x == 0) ALG_TRACE(0, 20);
  if (warp == 0) {  // one barrier per lane
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
  } else if (warp == 3) {
    // The table copies below run in different warps so that their first-touch misses (kernel
    // parameters, table in global memory) overlap instead of adding up.
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tmA) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tmB) : "memory");
    }
    for (int e = lane; e < q * q; e += 32) ctl->keep[e] = a.st.valid ? a.st.keep[e] : tab->keep[e];
  } else if (warp == 4) {
    if (a.dyn_so) asm volatile("griddepcontrol.wait;" ::: "memory");   // segment offsets written by the bucketing kernel
    for (int e = lane; e <= q; e += 32)
      ctl->so[e] = a.seg_rows ? e * a.seg_rows : a.dyn_so ? a.dyn_so[e] : a.st.valid ? a.st.so[e] : tab->so[e];
  } else if (warp == 5) {
    if (a.dyn_so) asm volatile("griddepcontrol.wait;" ::: "memory");
    for (int e = lane; e < q * q; e += 32) {
      const uint32_t mask = a.st.valid ? a.st.keep[e] : tab->keep[e];
      int n = 0;
      for (int k = 0; k < q; ++k)
        if ((mask >> k) & 1u)
          n += (a.seg_rows ? a.seg_rows
                : a.dyn_so   ? a.dyn_so[k + 1] - a.dyn_so[k]
                : a.st.valid ? a.st.so[k + 1] - a.st.so[k]
                             : tab->so[k + 1] - tab->so[k]) /
               BK;
      ctl->nkb[e] = (uint16_t)n;   // for tile records decoded after the precomputed ones
    }
  }
  if (threadIdx.x == 0) ALG_TRACE(0, 21);
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)),
                 "r"((uint32_t)C::kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // Programmatic dependent launch: everything above touches only this CTA's own state, so it may
  // run while the previous kernel of the stream is finishing; nothing below (bucket offsets, X, H,
  // Y) is read or written before that kernel has completed.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (warp == 2) {
    // one warp plans this CTA's work while the others set up barriers and tensor memory
    // cyclic schedule: planned on the host, once per (handle, M); the stamp in front of the records
    // tells whether the device copy still is the plan this launch was given
    bool planned = false;
    if (a.plan) {
      const TileRec stamp = a.plan[0];
      planned = stamp.row0 == a.M && stamp.rows == a.plan_tag;
    }
    if (planned) {
      for (int r = lane; r < a.plan_rounds; r += 32) recs[r] = a.plan[1 + (size_t)blockIdx.x * a.plan_stride + r];
      if (lane == 0) tm->seq_rounds = a.plan_rounds, tm->seq_valid = a.plan_rounds, tm->total = 0;
    } else {
      if (a.offsets || a.dyn_so) asm volatile("griddepcontrol.wait;" ::: "memory");  // bucket offsets come from the previous kernel
      tile_plan_warp(tm, recs, kSeqCap, tab, a.st, a.q, a.n_classes, a.offsets, a.cyclic_rows, a.M, a.geom, blockIdx.x,
                     gridDim.x, BK, a.dyn_so, a.seg_rows);
    }
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (threadIdx.x == 0) ALG_TRACE(0, 24);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;

  // The producer and MMA roles run warp-uniformly: all 32 lanes execute the loops and the waits,
  // and one elected lane issues the copy / MMA / commit instructions.  In a single-lane
  // (divergent) branch the compiler has to stage every operand of those instructions through
  // vector registers, which costs the issuing thread ~500 cycles per K block -- the whole budget
  // of a 128x256x64 block -- against ~290 cycles when the operands live in uniform registers.
  // Loop bounds read from shared memory are broadcast with a shuffle so that they count as
  // warp-uniform.
  if (warp == 0 || (AMODE == 2 ? warp >= kProducerWarpB : warp == kProducerWarpB)) {
    // ---------------- TMA producers: warp 0 loads A, the last warp loads B ----------------
    // Issuing a tiled load occupies the thread while the copy engine expands the box; with two
    // issuing warps a freed stage is refilled sooner, which shortens the
    // load -> MMA -> free -> load round trip that bounds the bytes in flight.
    const bool loads_a = warp == 0;
    int stage = 0, round = 0;
    uint32_t phase = 0;
    bool ok = true;
    const uint32_t full0 = smem_u32(&ctl->full[0]), empty0 = smem_u32(&ctl->empty[0]);
    const uint32_t smem0 = smem_u32(smem);
    TileRec rec = tile_seq_get(recs, tm, a.geom, 0, blockIdx.x, gridDim.x, ctl->nkb);
    while (ok && __shfl_sync(0xffffffffu, rec.row0, 0) >= 0) {
      ++round;
      if (loads_a && lane == 0) ALG_TRACE(0, 1);
      const int pair = __shfl_sync(0xffffffffu, rec.pair & 0xFFFF, 0);
      const int row0 = __shfl_sync(0xffffffffu, rec.row0, 0);
      const int n0 = __shfl_sync(0xffffffffu, rec.n0, 0);
      const uint32_t mask = __shfl_sync(0xffffffffu, ctl->keep[pair], 0);
      const int type_i = pair / q;
      const int a_row = a.a_cyclic_rows ? row0 - type_i * a.a_cyclic_rows : row0;
      // explicit types without a bucketed copy: a lane fetches four consecutive bucketed rows (and the same 128
      // rows further for 256-row tiles) through the permutation; rows past the batch repeat its last row, they
      // belong to no tile row that is stored
      // Issuing a gather costs its thread ~56 cycles and the lanes of a warp issue one after the other, so the 32
      // gathers of a 128-row stage are split between four warps (the two producers and two warps that do nothing
      // else): eight lanes each, warp w of the four takes rows 32 w .. 32 w + 31.
      int g_rows[TILE_M / 128][4];
      const int g_slot = (loads_a ? 0 : warp - kProducerWarpB + 1) * kGatherLanes + (lane & (kGatherLanes - 1));
      if (AMODE == 2) {
#pragma unroll
        for (int h = 0; h < TILE_M / 128; ++h)
#pragma unroll
          for (int j = 0; j < 4; ++j) g_rows[h][j] = __ldg(a.in_perm + min(row0 + h * 128 + g_slot * 4 + j, a.M - 1));
      }
      for (int k = 0; k < q && ok; ++k) {
        if (!((mask >> k) & 1u)) continue;
        const int k_begin = __shfl_sync(0xffffffffu, ctl->so[k], 0);
        const int k_end = __shfl_sync(0xffffffffu, ctl->so[k + 1], 0);
        for (int k0 = k_begin; k0 < k_end; k0 += BK) {
          ok = __all_sync(0xffffffffu, wait_bar(empty0 + 8u * (uint32_t)stage, phase ^ 1u, ctl, a.status));
          if (!ok) break;
          const uint32_t bar = full0 + 8u * (uint32_t)stage;
          const uint32_t sa = smem0 + (uint32_t)stage * (uint32_t)C::kStageBytes;
          if (AMODE == 2) {
            if (elect_one()) {
              if (loads_a) {
                mbar_expect_tx(bar, (uint32_t)C::kStageBytes);
              } else if (warp != kProducerWarpB) {
                // a gather-only warp
              } else if (GATED) {
                tma_load_3d(sa + C::kABytes, &tmB, bar, 0, k0, n0 >> 6);
                tma_load_3d(sa + C::kABytes + 2 * C::kBChunkBytes, &tmB, bar, 0, k0, (a.gated_f + n0) >> 6);
              } else if (a.b_3d) {
                tma_load_3d(sa + C::kABytes, &tmB, bar, 0, k0, n0 >> 6);
              } else {
#pragma unroll
                for (int c = 0; c < TILE_N / 64; ++c)
                  tma_load_2d(sa + C::kABytes + c * C::kBChunkBytes, &tmB, bar, n0 + c * 64, k0);
              }
            }
            __syncwarp();
            // one four-row gather per lane (and per 128 rows): 512 bytes each, 128-byte rows swizzled like a box
            if (lane < kGatherLanes) {
#pragma unroll
              for (int h = 0; h < TILE_M / 128; ++h)
                tma_gather4(sa + (uint32_t)(h * 128 * BK * 2 + g_slot * 4 * BK * 2), &tmA, bar, k0, g_rows[h][0], g_rows[h][1],
                            g_rows[h][2], g_rows[h][3]);
            }
          } else if (elect_one()) {
            if (a.seg_rows) {
              // weight gradient, cyclic schedule: rows k, k + q, ... of X (A, features contiguous) and of G (B),
              // 64 of them from position k0 - so[k] on, in boxes of 64 features / 64 output columns
              const int pos0 = k0 - k_begin;
              if (loads_a) {
                mbar_expect_tx(bar, (uint32_t)C::kStageBytes);
#pragma unroll
                for (int c = 0; c < TILE_M / 64; ++c) tma_load_3d(sa + c * (64 * BK * 2), &tmA, bar, row0 + c * 64, k, pos0);
              } else {
#pragma unroll
                for (int c = 0; c < TILE_N / 64; ++c)
                  tma_load_3d(sa + C::kABytes + c * C::kBChunkBytes, &tmB, bar, n0 + c * 64, k, pos0);
              }
            } else if (AMODE == 1 && loads_a && a.a_cyclic_rows) {
              // runs of run_rows rows per period: 64-row boxes, each inside one run
              mbar_expect_tx(bar, (uint32_t)C::kStageBytes);
#pragma unroll
              for (int h = 0; h < TILE_M / 64; ++h) {
                const int b = a_row + 64 * h, per = b / a.run_rows;
                tma_load_4d(sa + h * (64 * BK * 2), &tmA, bar, k0, b - per * a.run_rows, type_i, per);
              }
            } else if (loads_a) {
              mbar_expect_tx(bar, (uint32_t)C::kStageBytes);
              if (a.a_cyclic_rows) tma_load_3d(sa, &tmA, bar, k0, type_i, a_row);
              else tma_load_2d(sa, &tmA, bar, k0, a_row);
            } else if (a.w_kmajor) {
              // W used transposed: TILE_N rows of W (the output columns) x 64 of its columns (the reduction)
              tma_load_2d(sa + C::kABytes, &tmB, bar, k0, n0);
            } else if (GATED) {
              // two boxes of two 64-column chunks: the tile's gate columns, then its up columns
              tma_load_3d(sa + C::kABytes, &tmB, bar, 0, k0, n0 >> 6);
              tma_load_3d(sa + C::kABytes + 2 * C::kBChunkBytes, &tmB, bar, 0, k0, (a.gated_f + n0) >> 6);
            } else if (a.b_3d) {
              tma_load_3d(sa + C::kABytes, &tmB, bar, 0, k0, n0 >> 6);  // all 64-column chunks in one box
            } else {
#pragma unroll
              for (int c = 0; c < TILE_N / 64; ++c)
                tma_load_2d(sa + C::kABytes + c * C::kBChunkBytes, &tmB, bar, n0 + c * 64, k0);
            }
          }
          __syncwarp();
          if (++stage == C::kStages) stage = 0, phase ^= 1u;
        }
      }
      if (loads_a && lane == 0) ALG_TRACE(0, 2);
      rec = tile_seq_get(recs, tm, a.geom, round, blockIdx.x, gridDim.x, ctl->nkb);
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    int stage = 0, acc = 0, round = 0;
    uint32_t phase = 0, acc_phase = 0;
    bool ok = true;
    const uint32_t full0 = smem_u32(&ctl->full[0]), empty0 = smem_u32(&ctl->empty[0]);
    const uint32_t tfull0 = smem_u32(&ctl->tmem_full[0]), tempty0 = smem_u32(&ctl->tmem_empty[0]);
    // A: K-major rows of 128 (64) bytes; in the in-place weight-gradient pass the block lies MN-major like B
    // (64-feature chunks one box apart, 16 reduction rows = 128 descriptor units per K step)
    const uint64_t da0 = a.seg_rows ? make_smem_desc(smem_u32(smem), 64 * BK * 2, 1024)
                                    : make_smem_desc(smem_u32(smem), 16, C::kSboK, C::kSwzK);
    const uint64_t da_step = a.seg_rows ? 128 : 2;
    // B: the canonical bank lands MN-major (64-column chunks one box apart, 16 k-rows = two 8-row groups
    // = 128 descriptor units per K step); used transposed it lands K-major like A (32 bytes per K step)
    const uint64_t db0 = a.w_kmajor ? make_smem_desc(smem_u32(smem) + C::kABytes, 16, C::kSboK, C::kSwzK)
                                    : make_smem_desc(smem_u32(smem) + C::kABytes, C::kBChunkBytes, 1024);
    const uint32_t idesc = (a.w_kmajor ? (C::kIdesc & ~(1u << 16)) : C::kIdesc) | (a.seg_rows ? (1u << 15) : 0u);
    const uint64_t db_step = a.w_kmajor ? 2 : 128;
    TileRec rec = tile_seq_get(recs, tm, a.geom, 0, blockIdx.x, gridDim.x, ctl->nkb);
    while (ok && __shfl_sync(0xffffffffu, rec.row0, 0) >= 0) {
      ++round;
      if (lane == 0) ALG_TRACE(1, 1);
      // All kept products of the block run back to back into one accumulator, so this warp only
      // needs their total number of K blocks (upper half of rec.rows).
      const int n_kb = __shfl_sync(0xffffffffu, (int)((uint32_t)rec.rows >> 16), 0);
      ok = __all_sync(0xffffffffu, wait_bar(tempty0 + 8u * (uint32_t)acc, acc_phase ^ 1u, ctl, a.status));
      if (!ok) break;
      if (lane == 0) ALG_TRACE(1, 2);
      tc_fence_after();
      const uint32_t d_tmem = tmem_base + (uint32_t)(acc * C::kAccStride);
      for (int kb = 0; kb < n_kb; ++kb) {
        ok = __all_sync(0xffffffffu, wait_bar(full0 + 8u * (uint32_t)stage, phase, ctl, a.status));
        if (!ok) break;
        if (kb == 0 && lane == 0) ALG_TRACE(1, 3);
        tc_fence_after();
        const uint64_t da = da0 + (uint64_t)((uint32_t)stage * (uint32_t)(C::kStageBytes >> 4));
        const uint64_t db = db0 + (uint64_t)((uint32_t)stage * (uint32_t)(C::kStageBytes >> 4));
        if (elect_one()) {
          // A: 16 k-elements = 32 bytes inside the swizzle atom; B: 16 k-rows = two 8-row groups;
          // the second 128 rows of a 256-row tile sit behind the first in the stage and accumulate
          // TILE_N columns further in tensor memory
#pragma unroll
          for (int kk = 0; kk < BK / 16; ++kk)
#pragma unroll
            for (int h = 0; h < C::kHalves; ++h)
              tc_mma_bf16(d_tmem + (uint32_t)(h * TILE_N), da + (uint64_t)kk * da_step + (uint64_t)(h * (C::kAHalfBytes >> 4)), db + (uint64_t)kk * db_step,
                          idesc, (kb | kk) ? 1u : 0u);
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
      rec = tile_seq_get(recs, tm, a.geom, round, blockIdx.x, gridDim.x, ctl->nkb);
    }
  } else {
    // ---------------- epilogue: warp e handles TMEM lanes [32*(warp%4), +32), column half e/4 ----
    const int e = warp - 2;
    const int quad = warp & 3;
    const int half = e >> 2;
    int acc = 0, round = 0;
    uint32_t acc_phase = 0;
    TileRec rec = tile_seq_get(recs, tm, a.geom, 0, blockIdx.x, gridDim.x, ctl->nkb);
    while (rec.row0 >= 0) {
      ++round;
      const int r = (C::kHalves == 2 ? half * 128 : 0) + quad * 32 + lane;   // row of the tile this lane holds
      int64_t out_row = -1;
      const int tile_rows = rec.rows & 0xFFFF;
      // a tile without any K block (weight-gradient pass, row type absent from the batch): nothing was
      // accumulated, its result is zero
      const bool empty_tile = ((uint32_t)rec.rows >> 16) == 0u;
      if (r < tile_rows) {
        if (AMODE == 1 && a.out_cyclic_rows) {
          const int i = (rec.pair & 0xFFFF) / q;
          const int bt = rec.row0 + r - i * a.out_cyclic_rows, per = bt / a.run_rows;
          out_row = (int64_t)per * a.run_period + i * a.run_rows + (bt - per * a.run_rows);
        } else if (a.out_cyclic_rows) {
          const int i = (rec.pair & 0xFFFF) / q;
          out_row = (int64_t)(rec.row0 + r - i * a.out_cyclic_rows) * q + i;
        } else {
          out_row = a.perm ? __ldg(a.perm + rec.row0 + r) : (rec.row0 + r);
        }
        if (out_row >= a.M) out_row = -1;   // never store outside Y, whatever the tile record says
      }
      bool ok = wait_bar(smem_u32(&ctl->tmem_full[acc]), acc_phase, ctl, a.status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      if (e == 0 && lane == 0) ALG_TRACE(2, 1);
      tc_fence_after();
      const uint32_t taddr =
          tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * C::kAccStride + half * C::kHalf);
      const int col_base = rec.n0 + (C::kHalves == 2 ? 0 : half * C::kHalf);
      if (GATED) {
        // this warp: 32 rows x 64 output columns; gate values sit in accumulator columns [0, 128),
        // the matching up values 128 columns further
        const uint32_t tg = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * C::kAccStride + half * 64);
#pragma unroll 1
        for (int c0 = 0; c0 < 64; c0 += 32) {
          uint32_t vg[32], vu[32];
          tc_ld_32x32(tg + (uint32_t)c0, vg);
          tc_ld_32x32(tg + (uint32_t)(128 + c0), vu);
          tc_wait_ld();
          if (out_row >= 0) {
            float f[32];
#pragma unroll
            for (int x = 0; x < 32; ++x) {
              const float g = __uint_as_float(vg[x]);
              float th;
              asm("tanh.approx.f32 %0, %1;" : "=f"(th) : "f"(0.5f * g));
              f[x] = g * fmaf(0.5f, th, 0.5f) * __uint_as_float(vu[x]);   // silu(g) * u, sigmoid(g) = (1 + tanh(g/2)) / 2
            }
            finish_and_store_32(f, a, out_row, rec.n0 + half * 64 + c0);
          }
        }
      } else
      // bf16 outputs are transposed through a 2 KB staging buffer per warp: every lane writes its
      // own row segment (64 bytes, 16-byte pieces XOR-swizzled so that the writes and the reads
      // below are bank-conflict free), then four lanes together store one row segment, so one
      // store instruction covers 8 rows x 64 contiguous bytes (8 cache lines) instead of 32
      // lines with one sector each.  Works for every output addressing (bucketed, cyclic,
      // permuted) and for partial tiles.
      if (a.y_staged) {
        uint8_t *buf = store_buf + e * C::kStoreBufBytes;
        const uint32_t my_row = smem_u32(buf) + (uint32_t)lane * 64u;
        const uint32_t sw = (uint32_t)((lane >> 1) & 3);
        const int sub = lane >> 2, piece = lane & 3;   // row within a group of 8, 16-byte piece of the segment
        // destination rows of the four row groups this lane stores for (-1: beyond the tile)
        int64_t dst_row[4];
#pragma unroll
        for (int g = 0; g < 4; ++g) dst_row[g] = __shfl_sync(0xffffffffu, out_row, g * 8 + sub);
        const uint32_t rd_base = smem_u32(buf) + (uint32_t)sub * 64u;
#pragma unroll 1
        for (int c0 = 0; c0 < C::kHalf; c0 += 32) {
          uint32_t v[32];
          tc_ld_32x32(taddr + (uint32_t)c0, v);
          tc_wait_ld();
          float f[32];
#pragma unroll
          for (int x = 0; x < 32; ++x) f[x] = __uint_as_float(v[x]);
          if (empty_tile) {   // (rare and the same for the whole tile: a branch, not 32 selects per chunk)
#pragma unroll
            for (int x = 0; x < 32; ++x) f[x] = 0.f;
          }
          finish_32(f, a, col_base + c0);
          uint32_t w[16];
          pack_bf16_32(f, w);
          __syncwarp();  // the previous chunk has been read out of the buffer
#pragma unroll
          for (int g = 0; g < 4; ++g)
            asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(my_row + ((((uint32_t)g) ^ sw) << 4)), "r"(w[g * 4]),
                         "r"(w[g * 4 + 1]), "r"(w[g * 4 + 2]), "r"(w[g * 4 + 3])
                         : "memory");
          __syncwarp();
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            const int r = g * 8 + sub;                       // row of the chunk
            const uint32_t rsw = (uint32_t)((r >> 1) & 3);
            uint4 val;
            asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];"
                         : "=r"(val.x), "=r"(val.y), "=r"(val.z), "=r"(val.w)
                         : "r"(rd_base + (uint32_t)g * 512u + ((((uint32_t)piece) ^ rsw) << 4)));
            if (dst_row[g] >= 0)
              *(uint4 *)((__nv_bfloat16 *)a.Y + dst_row[g] * a.ldy + col_base + c0 + piece * 8) = val;
          }
        }
      } else {
#pragma unroll 1
      for (int c0 = 0; c0 < C::kHalf; c0 += 32) {
        uint32_t v[32];
        tc_ld_32x32(taddr + (uint32_t)c0, v);
        tc_wait_ld();
        if (out_row >= 0) {
          float f[32];
#pragma unroll
          for (int x = 0; x < 32; ++x) f[x] = __uint_as_float(v[x]);
          if (empty_tile) {
#pragma unroll
            for (int x = 0; x < 32; ++x) f[x] = 0.f;
          }
          finish_and_store_32(f, a, out_row, col_base + c0);
        }
      }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&ctl->tmem_empty[acc]));
      if (e == 0 && lane == 0) ALG_TRACE(2, 2);
      if (++acc == 2) acc = 0, acc_phase ^= 1u;
      rec = tile_seq_get(recs, tm, a.geom, round, blockIdx.x, gridDim.x, ctl->nkb);
    }
  }

  // ---------------- teardown ----------------
  __syncwarp();
  if (ctl->abort_flag) {
    // give copies that are still in flight time to land before shared memory is released
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000LL) {
    }
  }
  tc_fence_before();
  __syncthreads();
  ALG_TRACE_CTA(1, a.act ? 0 : 1);
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)C::kTmemCols)
                 : "memory");
  }
}

PFN_cuTensorMapEncodeTiled_v12000 g_encode = nullptr;

template <int TILE_N, int TILE_M, bool GATED, int BK, int AMODE = 0>
cudaError_t launch_bk(const ProjArgs &a, int num_sms, cudaStream_t st) {
  using C = Cfg<TILE_N, TILE_M, BK>;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(proj_tc_kernel<TILE_N, TILE_M, GATED, BK, AMODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  int smem_bytes = C::kFixedSmemBytes + (int)tile_map_bytes(a.n_classes);
  if (smem_bytes > 227 * 1024) return cudaErrorInvalidConfiguration;
  CUtensorMap tmA, tmB;
  cudaError_t e;
  ProjArgs b = a;
  if (a.seg_rows) {
    // X and G as {columns, type, position in the type}: rows t, t + q, ... are the reduction segment of type t
    if (GATED || a.w_kmajor || TILE_M != 128 || BK != 64) return cudaErrorInvalidValue;
    const uint64_t da[3] = {(uint64_t)a.M, (uint64_t)a.q, (uint64_t)a.seg_rows};
    const uint64_t sa[2] = {(uint64_t)a.ldx * 2, (uint64_t)a.ldx * 2 * (uint64_t)a.q};
    const uint64_t db[3] = {(uint64_t)a.N, (uint64_t)a.q, (uint64_t)a.seg_rows};
    const uint64_t sb[2] = {(uint64_t)a.ldw * 2, (uint64_t)a.ldw * 2 * (uint64_t)a.q};
    const uint32_t box[3] = {64, 1, 64};
    e = make_map_nd(&tmA, a.X, 3, da, sa, box, 128);
    if (e == cudaSuccess) e = make_map_nd(&tmB, a.W, 3, db, sb, box, 128);
    if (e != cudaSuccess) return e;
    b.b_3d = 0;
  } else {
  e = make_map_a(&tmA, a);
  if (e != cudaSuccess) return e;
  if (a.w_kmajor) {   // W is N x K here (rows = output columns, contiguous along the reduction): boxes of 64 x TILE_N
    if (GATED) return cudaErrorInvalidValue;
    b.b_3d = 0;
    e = make_map_2d_sw(&tmB, a.W, (uint64_t)a.K, (uint64_t)a.N, (uint64_t)a.ldw * 2, BK, TILE_N, BK * 2);
    if (e != cudaSuccess) return e;
  } else {
    b.b_3d = make_map_b3d(&tmB, a, GATED ? 2 : TILE_N / 64) == cudaSuccess;
  }
  if (GATED && !b.b_3d) return cudaErrorInvalidValue;
  if (!b.b_3d && !a.w_kmajor) {
    e = make_map_2d(&tmB, a.W, (uint64_t)a.N, (uint64_t)a.K, (uint64_t)a.ldw * 2, 64, BK);
    if (e != cudaSuccess) return e;
  }
  }
  // staging buffers for the transposing epilogue, when they fit and the output rows are 16-byte aligned
  b.y_staged = !GATED && a.y_bf16 && smem_bytes + kEpiWarps * C::kStoreBufBytes <= 227 * 1024 && ((uintptr_t)a.Y & 15u) == 0 &&
               (a.ldy * 2) % 16 == 0;
  if (b.y_staged) smem_bytes += kEpiWarps * C::kStoreBufBytes;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(num_sms, 1, 1);
  cfg.blockDim = dim3(AMODE == 2 ? kThreads + 32 * kGatherWarps : kThreads, 1, 1);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  e = cudaLaunchKernelEx(&cfg, proj_tc_kernel<TILE_N, TILE_M, GATED, BK, AMODE>, tmA, tmB, b);
  count_launch(1);
  return e;
}

template <int TILE_N, int TILE_M, bool GATED = false>
cudaError_t launch_t(const ProjArgs &a, int num_sms, cudaStream_t st) {
  // the in-place view of an interval schedule (runs of a type) is a kernel variant of its own, 64-deep stages only
  if (a.run_rows) return a.block_k == 64 ? launch_bk<TILE_N, TILE_M, GATED, 64, 1>(a, num_sms, st) : cudaErrorInvalidValue;
  // so are the rows of explicit types fetched through the permutation by the A producer
  if (a.in_perm) return a.block_k == 64 && !a.w_kmajor && !a.seg_rows ? launch_bk<TILE_N, TILE_M, GATED, 64, 2>(a, num_sms, st) : cudaErrorInvalidValue;
  if (a.block_k == 32) return launch_bk<TILE_N, TILE_M, GATED, 32>(a, num_sms, st);
  if (a.block_k == 64) return launch_bk<TILE_N, TILE_M, GATED, 64>(a, num_sms, st);
  return cudaErrorInvalidValue;
}

}  // namespace

namespace tc {
cudaError_t make_map_2d_sw(CUtensorMap *map, const void *base, uint64_t inner, uint64_t outer, uint64_t ld_bytes,
                           uint32_t box_inner, uint32_t box_outer, int swizzle_bytes) {
  cudaError_t e0 = tc_init();
  if (e0 != cudaSuccess) return e0;
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {ld_bytes};
  cuuint32_t box[2] = {box_inner, box_outer};
  cuuint32_t estr[2] = {1, 1};
  const CUtensorMapSwizzle sw = swizzle_bytes == 128  ? CU_TENSOR_MAP_SWIZZLE_128B
                                : swizzle_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                                : swizzle_bytes == 32 ? CU_TENSOR_MAP_SWIZZLE_32B
                                                      : CU_TENSOR_MAP_SWIZZLE_NONE;
  CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

cudaError_t make_map_nd(CUtensorMap *map, const void *base, int rank, const uint64_t *dims, const uint64_t *stride_bytes,
                        const uint32_t *box, int swizzle_bytes) {
  cudaError_t e0 = tc_init();
  if (e0 != cudaSuccess) return e0;
  if (rank < 2 || rank > 5) return cudaErrorInvalidValue;
  cuuint64_t d[5], st[4];
  cuuint32_t b[5], estr[5];
  for (int i = 0; i < rank; ++i) d[i] = dims[i], b[i] = box[i], estr[i] = 1;
  for (int i = 0; i + 1 < rank; ++i) st[i] = stride_bytes[i];
  const CUtensorMapSwizzle sw = swizzle_bytes == 128  ? CU_TENSOR_MAP_SWIZZLE_128B
                                : swizzle_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                                : swizzle_bytes == 32 ? CU_TENSOR_MAP_SWIZZLE_32B
                                                      : CU_TENSOR_MAP_SWIZZLE_NONE;
  CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void *>(base), d, st, b, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

cudaError_t make_map_2d(CUtensorMap *map, const void *base, uint64_t inner, uint64_t outer, uint64_t ld_bytes,
                        uint32_t box_inner, uint32_t box_outer) {
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {ld_bytes};
  cuuint32_t box[2] = {box_inner, box_outer};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

// The canonical K x N bank seen as {64 columns, K rows, N/64 column chunks}: one box of
// 64 x 64 x chunks lands in shared memory chunk-major ([chunk][k][64 n]), which is exactly the
// MN-major 128-byte-swizzled operand layout, with a single copy instruction per stage.
cudaError_t make_map_b3d(CUtensorMap *map, const ProjArgs &a, int chunks) {
  const int w_cols = a.gated_f ? 2 * a.gated_f : a.N;   // the merged gate/up bank is twice as wide as the output
  if (w_cols % 64) return cudaErrorInvalidValue;
  cuuint64_t dims[3] = {64, (cuuint64_t)a.K, (cuuint64_t)(w_cols / 64)};
  cuuint64_t strides[2] = {(cuuint64_t)a.ldw * 2, 128};
  cuuint32_t box[3] = {64, (cuuint32_t)a.block_k, (cuuint32_t)chunks};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(a.W), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

cudaError_t make_map_a(CUtensorMap *map, const ProjArgs &a) {
  const uint32_t box_rows = a.geom.tile_m == 256 && a.a_box_256 ? 256u : 128u;
  if (a.in_perm)   // rows fetched four at a time through the permutation: boxes of one row
    return make_map_2d_sw(map, a.X, (uint64_t)a.K, (uint64_t)a.M, (uint64_t)a.ldx * 2, (uint32_t)a.block_k, 1, a.block_k * 2);
  if (!a.a_cyclic_rows)
    return make_map_2d_sw(map, a.X, (uint64_t)a.K, (uint64_t)a.M, (uint64_t)a.ldx * 2, (uint32_t)a.block_k, box_rows,
                          a.block_k * 2);
  if (a.run_rows) {   // {K, row in run, type, period}, boxes of 64 rows
    const uint64_t dims[4] = {(uint64_t)a.K, (uint64_t)a.run_rows, (uint64_t)a.q, (uint64_t)(a.M / a.run_period)};
    const uint64_t str[3] = {(uint64_t)a.ldx * 2, (uint64_t)a.ldx * 2 * (uint64_t)a.run_rows, (uint64_t)a.ldx * 2 * (uint64_t)a.run_period};
    const uint32_t box[4] = {(uint32_t)a.block_k, 64, 1, 1};
    return make_map_nd(map, a.X, 4, dims, str, box, a.block_k * 2);
  }
  cuuint64_t dims[3] = {(cuuint64_t)a.K, (cuuint64_t)a.q, (cuuint64_t)a.a_cyclic_rows};
  cuuint64_t strides[2] = {(cuuint64_t)a.ldx * 2, (cuuint64_t)a.ldx * 2 * (cuuint64_t)a.q};
  cuuint32_t box[3] = {(cuuint32_t)a.block_k, 1, box_rows};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(a.X), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, a.block_k == 32 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

}  // namespace tc

cudaError_t tc_init() {
  if (g_encode) return cudaSuccess;
  void *fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
  if (e != cudaSuccess) return e;
  if (qres != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
  g_encode = (PFN_cuTensorMapEncodeTiled_v12000)fn;
  return cudaSuccess;
}

cudaError_t launch_proj_tc_gated(const ProjArgs &a, int num_sms, cudaStream_t st) {
  cudaError_t e = tc_init();
  if (e != cudaSuccess) return e;
  if (!a.gated_f || a.geom.tile_m != 128 || !a.y_bf16) return cudaErrorInvalidValue;
  return launch_t<256, 128, true>(a, num_sms, st);
}

cudaError_t launch_proj_tc(const ProjArgs &a, int tile_n, int num_sms, cudaStream_t st) {
  cudaError_t e = tc_init();
  if (e != cudaSuccess) return e;
  if (a.geom.tile_m == 256) {
    if (tile_n != 128) return cudaErrorInvalidValue;
    ProjArgs b = a;
    b.a_box_256 = 1;   // one box brings all 256 rows of a stage
    return launch_t<128, 256>(b, num_sms, st);
  }
  if (tile_n == 256) return launch_t<256, 128>(a, num_sms, st);
  if (tile_n == 192) return launch_t<192, 128>(a, num_sms, st);
  if (tile_n == 128) return launch_t<128, 128>(a, num_sms, st);
  return cudaErrorInvalidValue;
}

}  // namespace algproj
