// The two-map FFN  Y = (act(X *_q W_up + b_up)) *_q W_down + b_down  as ONE persistent kernel
// (cyclic schedule, bf16, q <= 8).
//
// The two projections are the grouped tcgen05 GEMM of proj_tc.cu (same tiles, same operand
// layouts, same accumulation of all kept products of a block in one TMEM accumulator, Eqs.
// typed-diag/off).  Run as two kernels, every boundary costs each SM ~9 k cycles without tensor
// work (last epilogue, prologue, first operands from DRAM) and the down projection has only 1.7
// tiles per CTA to balance.  Here every CTA walks one host-planned list that holds up tiles and
// down tiles:
//   * an up tile (128 rows of one type x 256 columns of one hidden group) ends with its rows of H
//     stored in bucketed order; a signal warp then publishes it: device-scope fence + one atomic
//     add on the counter of (row block, hidden group);
//   * a down tile (the same 128 rows x 256, 192 or 128 output columns) reads H one kept hidden
//     group after the other; before the loads of a group it waits until that group's counter has
//     reached the number of up tiles of the group.
// The planner (api.cu) list-schedules the tiles on the host: up tiles first, row block by row
// block, then down tiles longest first as they become ready, in a simulated timeline; a list that
// is valid in a simulated timeline cannot deadlock (a wait cycle would need two down tiles that
// each start before the other).  All CTAs are co-resident (one per SM, grid <= SM count), every
// wait is bounded, and on expiry the CTA raises ALG_ERR_DEVICE_TIMEOUT and leaves.
//
// Warp roles (384 threads): 0 = TMA producer of A, 10 = TMA producer of B, 1 = TMEM allocator and
// MMA issuer, 2..9 = epilogue, 11 = signal warp.  Producer and MMA warps run warp-uniformly with
// one elected issuing lane (see proj_tc.cu).
#include <cudaTypedefs.h>

#include <cstdlib>
#include <cstring>

#include "tc_common.cuh"

namespace algproj {

using namespace tc;

namespace {

constexpr int kEpiWarps = 8;
constexpr int kProducerWarpB = 2 + kEpiWarps;
constexpr int kSignalWarp = 3 + kEpiWarps;
constexpr int kThreads = 32 * (4 + kEpiWarps);
constexpr int kStages = 4;
constexpr int kABytes = kTcTileM * kTcBlockK * 2;   // 16 KB
constexpr int kBChunkBytes = kTcBlockK * 64 * 2;     // 8 KB: one 64(k) x 64(n) box
constexpr int kStageBytes = kABytes + 4 * kBChunkBytes;
constexpr int kAccStride = 256;
constexpr int kTmemCols = 512;
constexpr int kStoreBufBytes = 32 * 64;

struct Ctl {
  uint64_t full[kStages];
  uint64_t empty[kStages];
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint32_t tmem_base;
  volatile int abort_flag;
  volatile int stored;   // epilogue warps that have finished storing an up tile (running total)
  int pad;
};
constexpr int kSmemBytes = kStages * kStageBytes + kEpiWarps * kStoreBufBytes + (int)sizeof(Ctl) +
                           kFfnSeqCap * (int)(sizeof(TileRec) + sizeof(TileExt)) + 1024;
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");

__device__ __noinline__ bool wait_slow(uint32_t bar, uint32_t parity, Ctl *ctl, int *status) {
  const long long t0 = clock64();
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 255u) == 0) {
      if (ctl->abort_flag) return false;
      if (clock64() - t0 > kTimeoutCycles) {
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


#ifdef ALGPROJ_TRACE
#define FTRACE(role, tag)                                                                                     \
  do {                                                                                                        \
    const unsigned tr_cta = blockIdx.x - (unsigned)(fa.p[0].dbg >> 8);                                        \
    if (fa.p[0].trace && tr_cta < 8u && tr_n < fa.p[0].trace_cap)                                             \
      fa.p[0].trace[((size_t)tr_cta * 3 + (role)) * fa.p[0].trace_cap + tr_n++] = (clock64() << 8) | (tag);   \
  } while (0)
#else
#define FTRACE(role, tag) \
  do {                    \
  } while (0)
#endif

__global__ void __launch_bounds__(kThreads, 1)
ffn_tc_kernel(const __grid_constant__ CUtensorMap tmA_up, const __grid_constant__ CUtensorMap tmB_up,
              const __grid_constant__ CUtensorMap tmA_dn, const __grid_constant__ CUtensorMap tmB_dn,
              const __grid_constant__ CUtensorMap tmB_dn3, const __grid_constant__ CUtensorMap tmB_dn_half,
              const __grid_constant__ FfnArgs fa) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t *store_buf = smem + kStages * kStageBytes;
  Ctl *ctl = (Ctl *)(store_buf + kEpiWarps * kStoreBufBytes);
  TileRec *recs = (TileRec *)(ctl + 1);
  TileExt *exts = (TileExt *)(recs + kFfnSeqCap);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int *status = fa.p[0].status;
  [[maybe_unused]] int tr_n = 0;
#ifdef ALGPROJ_TRACE
  if (fa.p[0].trace && threadIdx.x == 0) {  // whole-CTA window: global timer and SM clock at entry
    unsigned long long gt;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(gt));
    fa.p[0].trace[(size_t)24 * fa.p[0].trace_cap + blockIdx.x * 4 + 0] = (long long)gt;
    fa.p[0].trace[(size_t)24 * fa.p[0].trace_cap + blockIdx.x * 4 + 2] = clock64();
  }
#endif

  if (warp == 0) {  // one barrier per lane
    if (lane < kStages) {
      mbar_init(smem_u32(&ctl->full[lane]), 1);
      mbar_init(smem_u32(&ctl->empty[lane]), 1);
    } else if (lane < kStages + 2) {
      mbar_init(smem_u32(&ctl->tmem_full[lane - kStages]), 1);
      mbar_init(smem_u32(&ctl->tmem_empty[lane - kStages]), kEpiWarps);
    } else if (lane == 31) {
      ctl->abort_flag = 0;
      ctl->stored = 0;
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  } else if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)),
                 "r"((uint32_t)kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  } else if (warp == 2) {
    for (int r = lane; r < fa.plan_rounds; r += 32) {
      recs[r] = fa.plan[(size_t)blockIdx.x * fa.plan_stride + r];
      exts[r] = fa.ext[(size_t)blockIdx.x * fa.plan_stride + r];
    }
  } else if (warp == 3 && lane < 6) {
    const CUtensorMap *maps[6] = {&tmA_up, &tmB_up, &tmA_dn, &tmB_dn, &tmB_dn3, &tmB_dn_half};
    asm volatile("prefetch.tensormap [%0];" ::"l"(maps[lane]) : "memory");
  }
  // Programmatic dependent launch: everything above touches only this CTA's own state and the plan
  // (written before the stream reached this launch).
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;

  if (warp == 0 || warp == kProducerWarpB) {
    // ---------------- TMA producers: warp 0 loads A (X or H), warp 10 loads B (W_up or W_down) ------
    const bool loads_a = warp == 0;
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    const uint32_t full0 = smem_u32(&ctl->full[0]), empty0 = smem_u32(&ctl->empty[0]);
    const uint32_t smem0 = smem_u32(smem);
    for (int pos = 0; ok; ++pos) {
      const TileRec rec = recs[pos];
      const int row0 = __shfl_sync(0xffffffffu, rec.row0, 0);
      if (row0 < 0) break;
      const int dep = __shfl_sync(0xffffffffu, exts[pos].dep, 0);
      const bool down = dep >= 0;
      const ProjArgs &a = fa.p[down ? 1 : 0];
      const int q = a.q;
      const int pair = __shfl_sync(0xffffffffu, rec.pair & 0xFFFF, 0);
      const int cols = __shfl_sync(0xffffffffu, rec.pair >> 16, 0);
      const int n0 = __shfl_sync(0xffffffffu, rec.n0, 0);
      const uint32_t mask = a.st.keep[pair];
      const int type_i = pair / q;
      const int a_row = a.a_cyclic_rows ? row0 - type_i * a.a_cyclic_rows : row0;
      const uint32_t tx_bytes = (uint32_t)(kABytes + (cols >> 6) * kBChunkBytes);
      if (loads_a && lane == 0) FTRACE(0, down ? 5 : 1);
      for (int k = 0; k < q && ok; ++k) {
        if (!((mask >> k) & 1u)) continue;
        const int k_begin = a.st.so[k], k_end = a.st.so[k + 1];
        if (down && loads_a) {
          // hidden group k of these rows of H must be complete: wait for the counter of (row block, k).
          // The other kept group of the tile is awaited only when the K loop reaches it, so its
          // hand-over hides behind the MMAs of this one.
          if (lane == 0) {
            const unsigned long long *cnt = fa.counters + (size_t)dep * q + k;
            const unsigned long long need = (unsigned long long)fa.target[k];
            const long long t0 = clock64();
            unsigned long long seen;
            while (true) {
              asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(seen) : "l"(cnt) : "memory");
              if (seen >= need) break;
              __nanosleep(100);
              if (ctl->abort_flag || clock64() - t0 > kTimeoutCycles) {
                ctl->abort_flag = 1;
                atomicExch(status, (int)ALG_ERR_DEVICE_TIMEOUT);
                ok = false;
                break;
              }
            }
            // H was written through the generic proxy by other SMs and is read by the copy engine
            asm volatile("fence.proxy.async;" ::: "memory");
            FTRACE(0, 6);
          }
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
        }
        for (int k0 = k_begin; k0 < k_end; k0 += kTcBlockK) {
          ok = __all_sync(0xffffffffu, wait_bar(empty0 + 8u * (uint32_t)stage, phase ^ 1u, ctl, status));
          if (!ok) break;
          const uint32_t bar = full0 + 8u * (uint32_t)stage;
          const uint32_t sa = smem0 + (uint32_t)stage * (uint32_t)kStageBytes;
          if (elect_one()) {
            if (loads_a) {
              mbar_expect_tx(bar, tx_bytes);
              if (down) tma_load_2d(sa, &tmA_dn, bar, k0, a_row);
              else if (a.a_cyclic_rows) tma_load_3d(sa, &tmA_up, bar, k0, type_i, a_row);
              else tma_load_2d(sa, &tmA_up, bar, k0, a_row);
            } else if (!down) {
              tma_load_3d(sa + kABytes, &tmB_up, bar, 0, k0, n0 >> 6);
            } else if (cols == 256) {
              tma_load_3d(sa + kABytes, &tmB_dn, bar, 0, k0, n0 >> 6);
            } else if (cols == 192) {
              tma_load_3d(sa + kABytes, &tmB_dn3, bar, 0, k0, n0 >> 6);
            } else {
              tma_load_3d(sa + kABytes, &tmB_dn_half, bar, 0, k0, n0 >> 6);
            }
          }
          __syncwarp();
          if (++stage == kStages) stage = 0, phase ^= 1u;
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
    const uint64_t da0 = make_smem_desc(smem_u32(smem), 16, 1024);
    const uint64_t db0 = make_smem_desc(smem_u32(smem) + kABytes, kBChunkBytes, 1024);
    for (int pos = 0; ok; ++pos) {
      const TileRec rec = recs[pos];
      if (__shfl_sync(0xffffffffu, rec.row0, 0) < 0) break;
      const int n_kb = __shfl_sync(0xffffffffu, (int)((uint32_t)rec.rows >> 16), 0);
      const int cols = __shfl_sync(0xffffffffu, rec.pair >> 16, 0);
      // instruction descriptor: D=f32, A=B=bf16, A K-major, B MN-major, N = cols, M = 128
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | (1u << 16) |
                             ((uint32_t)(cols >> 3) << 17) | ((uint32_t)(kTcTileM >> 4) << 24);
      ok = __all_sync(0xffffffffu, wait_bar(tempty0 + 8u * (uint32_t)acc, acc_phase ^ 1u, ctl, status));
      if (!ok) break;
      tc_fence_after();
      const uint32_t d_tmem = tmem_base + (uint32_t)(acc * kAccStride);
      for (int kb = 0; kb < n_kb; ++kb) {
        ok = __all_sync(0xffffffffu, wait_bar(full0 + 8u * (uint32_t)stage, phase, ctl, status));
        if (!ok) break;
        if (kb == 0 && lane == 0) FTRACE(1, cols == 256 ? 3 : 7);
        tc_fence_after();
        const uint64_t da = da0 + (uint64_t)((uint32_t)stage * (uint32_t)(kStageBytes >> 4));
        const uint64_t db = db0 + (uint64_t)((uint32_t)stage * (uint32_t)(kStageBytes >> 4));
        if (elect_one()) {
          tc_mma_bf16(d_tmem, da, db, idesc, kb ? 1u : 0u);
#pragma unroll
          for (int kk = 1; kk < kTcBlockK / 16; ++kk)
            tc_mma_bf16(d_tmem, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 128), idesc, 1u);
          tc_commit(empty0 + 8u * (uint32_t)stage);
        }
        __syncwarp();
        if (++stage == kStages) stage = 0, phase ^= 1u;
      }
      if (!ok) break;
      if (elect_one()) tc_commit(tfull0 + 8u * (uint32_t)acc);
      __syncwarp();
      if (lane == 0) FTRACE(1, 4);
      if (++acc == 2) acc = 0, acc_phase ^= 1u;
    }
  }
  else if (warp >= 2 && warp < 2 + kEpiWarps) {
    // ---------------- epilogue: warp e handles TMEM lanes [32*(warp%4), +32), column half e/4 ----
    const int e = warp - 2;
    const int quad = warp & 3;
    const int half = e >> 2;
    int acc = 0;
    uint32_t acc_phase = 0;
    uint8_t *buf = store_buf + e * kStoreBufBytes;
    const uint32_t my_row = smem_u32(buf) + (uint32_t)lane * 64u;
    const uint32_t sw = (uint32_t)((lane >> 1) & 3);
    const int sub = lane >> 2, piece = lane & 3;
    const uint32_t rd_base = smem_u32(buf) + (uint32_t)sub * 64u;
    for (int pos = 0;; ++pos) {
      const TileRec rec = recs[pos];
      if (rec.row0 < 0) break;
      const bool down = exts[pos].dep >= 0;
      const ProjArgs &a = fa.p[down ? 1 : 0];
      const int q = a.q;
      const int cols = rec.pair >> 16;
      const int cols_half = cols >> 1;
      const int r = quad * 32 + lane;
      int64_t out_row = -1;
      if (r < (rec.rows & 0xFFFF)) {
        if (a.out_cyclic_rows) {
          const int i = (rec.pair & 0xFFFF) / q;
          out_row = (int64_t)(rec.row0 + r - i * a.out_cyclic_rows) * q + i;
        } else {
          out_row = rec.row0 + r;
        }
      }
      bool ok = wait_bar(smem_u32(&ctl->tmem_full[acc]), acc_phase, ctl, status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      if (e == 0 && lane == 0) FTRACE(2, 1);
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * kAccStride + half * cols_half);
      const int col_base = rec.n0 + half * cols_half;
      int64_t dst_row[4];
#pragma unroll
      for (int g = 0; g < 4; ++g) dst_row[g] = __shfl_sync(0xffffffffu, out_row, g * 8 + sub);
#pragma unroll 1
      for (int c0 = 0; c0 < cols_half; c0 += 32) {
        uint32_t v[32];
        tc_ld_32x32(taddr + (uint32_t)c0, v);
        tc_wait_ld();
        float f[32];
#pragma unroll
        for (int x = 0; x < 32; ++x) f[x] = __uint_as_float(v[x]);
        if (!a.y_bf16) {  // fp32 result (final output only): direct 32-byte stores
          if (out_row >= 0) finish_and_store_32(f, a, out_row, col_base + c0);
          continue;
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
          const int rr = g * 8 + sub;
          const uint32_t rsw = (uint32_t)((rr >> 1) & 3);
          uint4 val;
          asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];"
                       : "=r"(val.x), "=r"(val.y), "=r"(val.z), "=r"(val.w)
                       : "r"(rd_base + (uint32_t)g * 512u + ((((uint32_t)piece) ^ rsw) << 4)));
          if (dst_row[g] >= 0)
            *(uint4 *)((__nv_bfloat16 *)a.Y + dst_row[g] * a.ldy + col_base + c0 + piece * 8) = val;
        }
      }
      tc_fence_before();
      __syncwarp();
      if (e == 0 && lane == 0) FTRACE(2, 2);
      if (lane == 0) {
        mbar_arrive(smem_u32(&ctl->tmem_empty[acc]));
        if (!down) {  // this warp's part of the H tile is stored: tell the signal warp
          __threadfence_block();
          atomicAdd((int *)&ctl->stored, 1);
        }
      }
      if (++acc == 2) acc = 0, acc_phase ^= 1u;
    }
  } else if (warp == kSignalWarp) {
    // ---------------- signal warp: publishes finished up tiles to the other CTAs ----------------
    if (lane == 0) {
      int n_up = 0;
      for (int pos = 0;; ++pos) {
        const TileRec rec = recs[pos];
        if (rec.row0 < 0) break;
        const int sig = exts[pos].sig;
        if (sig < 0) continue;
        ++n_up;
        const long long t0 = clock64();
        bool ok = true;
        while (ctl->stored < n_up * kEpiWarps) {
          __nanosleep(200);
          if (ctl->abort_flag || clock64() - t0 > kTimeoutCycles) {
            ctl->abort_flag = 1;
            atomicExch(status, (int)ALG_ERR_DEVICE_TIMEOUT);
            ok = false;
            break;
          }
        }
        if (!ok) break;
        // the epilogue warps' stores happen-before their counter increments (block-scope fence);
        // this device-scope fence makes them visible before the row block's counter moves
        __threadfence();
        atomicAdd(fa.counters + sig, 1ull);
      }
    }
  }

  // ---------------- teardown ----------------
  __syncwarp();
  if (ctl->abort_flag) {
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000LL) {
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kTmemCols)
                 : "memory");
  }
#ifdef ALGPROJ_TRACE
  if (fa.p[0].trace && threadIdx.x == 0) {
    unsigned long long gt;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(gt));
    fa.p[0].trace[(size_t)24 * fa.p[0].trace_cap + blockIdx.x * 4 + 1] = (long long)gt;
    fa.p[0].trace[(size_t)24 * fa.p[0].trace_cap + blockIdx.x * 4 + 3] = clock64();
  }
#endif
  // The last CTA to leave clears the counters for the next launch (which reads them only after
  // this kernel has completed), so a launch recorded in a CUDA graph replays correctly.
  if (threadIdx.x == 0) {
    __threadfence();
    const unsigned long long left = atomicAdd(fa.counters + fa.n_counters, 1ull);
    if (left == (unsigned long long)gridDim.x - 1) {
      for (int b = 0; b <= fa.n_counters; ++b) fa.counters[b] = 0;
      __threadfence();
    }
  }
}

}  // namespace

// Tensor maps: A of the up projection (X: plain rows or the type-strided cyclic view), A of the
// down projection (H in bucketed row order), B of both (3-D chunked views of the canonical banks;
// W_down also with a two-chunk box for 128-wide tiles).
cudaError_t launch_ffn_tc(const FfnArgs &fa, int n_workers, cudaStream_t st) {
  cudaError_t e = tc_init();
  if (e != cudaSuccess) return e;
  static bool attr_set = false;
  if (!attr_set) {
    e = cudaFuncSetAttribute(ffn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  CUtensorMap tmA_up, tmB_up, tmA_dn, tmB_dn, tmB_dn3, tmB_dn_half;
  if ((e = make_map_a(&tmA_up, fa.p[0])) != cudaSuccess) return e;
  if ((e = make_map_b3d(&tmB_up, fa.p[0], 4)) != cudaSuccess) return e;
  if ((e = make_map_a(&tmA_dn, fa.p[1])) != cudaSuccess) return e;
  if ((e = make_map_b3d(&tmB_dn, fa.p[1], 4)) != cudaSuccess) return e;
  if ((e = make_map_b3d(&tmB_dn3, fa.p[1], 3)) != cudaSuccess) return e;
  if ((e = make_map_b3d(&tmB_dn_half, fa.p[1], 2)) != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_workers, 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = std::getenv("ALGPROJ_NO_PDL") ? 0 : 1;
  e = cudaLaunchKernelEx(&cfg, ffn_tc_kernel, tmA_up, tmB_up, tmA_dn, tmB_dn, tmB_dn3, tmB_dn_half, fa);
  count_launch(1);
  return e;
}

}  // namespace algproj
