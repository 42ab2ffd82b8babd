// Grouped bf16 GEMM over the interaction table for sm_100a: TMA-fed shared-memory tiles,
// tcgen05.mma with the accumulator in tensor memory, persistent CTAs walking the tile
// enumeration (tile_map.cuh) in a static boustrophedon order.
//
// One output tile = 128 rows of one row type i  x  TILE_N columns of one output group j.  All
// kept products of that block (x_k W_kj for k in B(i,j); Eq. recursive-row-action -- for the
// Q_q law x_i W_ij + x_j W_jj, Eqs. typed-diag/off) are issued back to back into the SAME
// TMEM accumulator, so no partial sum ever reaches HBM ("one forward kernel accumulates both
// endpoint products before writing the output", Section "Kernels").
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

#include <cstdlib>

#include "tc_common.cuh"

namespace algproj {

using namespace tc;

namespace {

struct Ctl {
  uint64_t full[8];
  uint64_t empty[8];
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint32_t tmem_base;
  volatile int abort_flag;
  // interaction table, copied once per CTA so no role waits on global metadata at a tile start
  int so[kMaxQ + 1];
  uint32_t keep[kMaxPairs];
};

// Bounded wait. Returns false when the CTA is aborting.
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

constexpr int kSeqCap = 224;  // precomputed tile records per CTA
#ifndef ALGPROJ_EPI_WARPS
#define ALGPROJ_EPI_WARPS 8
#endif
constexpr int kEpiWarps = ALGPROJ_EPI_WARPS;
constexpr int kProducerWarpB = 2 + kEpiWarps;   // second TMA producer, after the epilogue warps
constexpr int kThreads = 32 * (3 + kEpiWarps);

template <int TILE_N>
struct Cfg {
  static constexpr int kABytes = kTcTileM * kTcBlockK * 2;      // 16 KB
  static constexpr int kBChunkBytes = kTcBlockK * 64 * 2;       // one 64(k) x 64(n) box: 8 KB
  static constexpr int kBBytes = kBChunkBytes * (TILE_N / 64);
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kStages = (200 * 1024) / kStageBytes > 8 ? 8 : (200 * 1024) / kStageBytes;
  static constexpr int kAccStride = TILE_N <= 128 ? 128 : 256;   // TMEM columns between the two accumulators
  static constexpr int kTmemCols = 2 * kAccStride;
  static constexpr int kFixedSmemBytes = kStages * kStageBytes + (int)sizeof(Ctl) + kSeqCap * 16 + 16 + 1024;  // + tile map
  static constexpr int kHalf = TILE_N / (kEpiWarps / 4);          // columns per epilogue warp
  // instruction descriptor: D=f32, A=B=bf16, A K-major, B MN-major, N, M=128
  static constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | (1u << 16) |
                                     ((uint32_t)(TILE_N >> 3) << 17) | ((uint32_t)(kTcTileM >> 4) << 24);
};

template <int TILE_N>
__global__ void __launch_bounds__(kThreads, 1)
proj_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const ProjArgs a) {
  using C = Cfg<TILE_N>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  Ctl *ctl = (Ctl *)(smem + C::kStages * C::kStageBytes);
  TileRec *recs = (TileRec *)(ctl + 1);
  TileMap *tm = (TileMap *)(recs + kSeqCap);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const DevTable *__restrict__ tab = a.tab;
  const int q = a.q;
  [[maybe_unused]] int tr_n = 0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::kStages; ++s) {
      mbar_init(smem_u32(&ctl->full[s]), 1);
      mbar_init(smem_u32(&ctl->empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&ctl->tmem_full[b]), 1);
      mbar_init(smem_u32(&ctl->tmem_empty[b]), kEpiWarps);
    }
    ctl->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmA) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmB) : "memory");
  }
  for (int e = threadIdx.x; e < q * q; e += kThreads) ctl->keep[e] = a.st.valid ? a.st.keep[e] : tab->keep[e];
  for (int e = threadIdx.x; e <= q; e += kThreads) ctl->so[e] = a.st.valid ? a.st.so[e] : tab->so[e];
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
  asm volatile("griddepcontrol.wait;" ::: "memory");
  tile_map_build(tm, tab, a.st, a.q, a.n_classes, a.offsets, a.cyclic_rows, a.M, a.geom);
  tile_seq_build(recs, kSeqCap, tm, a.geom, blockIdx.x, gridDim.x);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;

  if (warp == 0 || warp == kProducerWarpB) {
    // ---------------- TMA producers (one lane each): warp 0 loads A, the last warp loads B ----------------
    // Issuing a tiled load occupies the thread while the copy engine expands the box; with two
    // issuing threads a freed stage is refilled sooner, which shortens the
    // load -> MMA -> free -> load round trip that bounds the bytes in flight.
    if (lane == 0) {
      const bool loads_a = warp == 0;
      int stage = 0, round = 0;
      uint32_t phase = 0;
      bool ok = true;
      TileRec rec = tile_seq_get(recs, kSeqCap, tm, a.geom, 0, blockIdx.x, gridDim.x);
      while (ok && rec.row0 >= 0) {
        ++round;
        if (loads_a) ALG_TRACE(0, 1);
        const uint32_t mask = ctl->keep[rec.pair & 0xFFFF];
        const int type_i = (rec.pair & 0xFFFF) / q;
        const int a_row = a.a_cyclic_rows ? rec.row0 - type_i * a.a_cyclic_rows : rec.row0;
        for (int k = 0; k < q && ok; ++k) {
          if (!((mask >> k) & 1u)) continue;
          const int k_end = ctl->so[k + 1];
          for (int k0 = ctl->so[k]; k0 < k_end; k0 += kTcBlockK) {
            ok = wait_bar(smem_u32(&ctl->empty[stage]), phase ^ 1u, ctl, a.status);
            if (!ok) break;
            const uint32_t bar = smem_u32(&ctl->full[stage]);
            const uint32_t sa = smem_u32(smem + stage * C::kStageBytes);
            if (loads_a) {
              mbar_expect_tx(bar, (uint32_t)C::kStageBytes);
              if (a.a_cyclic_rows) tma_load_3d(sa, &tmA, bar, k0, type_i, a_row);
              else tma_load_2d(sa, &tmA, bar, k0, a_row);
            } else if (a.b_3d) {
              tma_load_3d(sa + C::kABytes, &tmB, bar, 0, k0, rec.n0 >> 6);  // all 64-column chunks in one box
            } else {
#pragma unroll
              for (int c = 0; c < TILE_N / 64; ++c)
                tma_load_2d(sa + C::kABytes + c * C::kBChunkBytes, &tmB, bar, rec.n0 + c * 64, k0);
            }
            if (++stage == C::kStages) stage = 0, phase ^= 1u;
          }
        }
        if (loads_a) ALG_TRACE(0, 2);
        rec = tile_seq_get(recs, kSeqCap, tm, a.geom, round, blockIdx.x, gridDim.x);
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer (one lane) ----------------
    if (lane == 0) {
      int stage = 0, acc = 0, round = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      TileRec rec = tile_seq_get(recs, kSeqCap, tm, a.geom, 0, blockIdx.x, gridDim.x);
      while (ok && rec.row0 >= 0) {
        ++round;
        ALG_TRACE(1, 1);
        ok = wait_bar(smem_u32(&ctl->tmem_empty[acc]), acc_phase ^ 1u, ctl, a.status);
        if (!ok) break;
        ALG_TRACE(1, 2);
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * C::kAccStride);
        const uint32_t mask = ctl->keep[rec.pair & 0xFFFF];
        uint32_t accumulate = 0;
        for (int k = 0; k < q && ok; ++k) {
          if (!((mask >> k) & 1u)) continue;
          const int n_kb = (ctl->so[k + 1] - ctl->so[k]) / kTcBlockK;
          for (int kb = 0; kb < n_kb; ++kb) {
            ok = wait_bar(smem_u32(&ctl->full[stage]), phase, ctl, a.status);
            if (!ok) break;
            if (!accumulate) ALG_TRACE(1, 3);
            tc_fence_after();
            const uint32_t sa = smem_u32(smem + stage * C::kStageBytes);
            const uint64_t da = make_smem_desc(sa, 16, 1024);
            const uint64_t db = make_smem_desc(sa + C::kABytes, C::kBChunkBytes, 1024);
#pragma unroll
            for (int kk = 0; kk < kTcBlockK / 16; ++kk) {
              // A: 16 k-elements = 32 bytes inside the swizzle atom; B: 16 k-rows = two 8-row groups
              tc_mma_bf16(d_tmem, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 128), C::kIdesc, accumulate);
              accumulate = 1;
            }
            tc_commit(smem_u32(&ctl->empty[stage]));
            if (++stage == C::kStages) stage = 0, phase ^= 1u;
          }
        }
        if (!ok) break;
        tc_commit(smem_u32(&ctl->tmem_full[acc]));
        ALG_TRACE(1, 4);
        if (++acc == 2) acc = 0, acc_phase ^= 1u;
        rec = tile_seq_get(recs, kSeqCap, tm, a.geom, round, blockIdx.x, gridDim.x);
      }
    }
  } else {
    // ---------------- epilogue: warp e handles TMEM lanes [32*(warp%4), +32), column half e/4 ----
    const int e = warp - 2;
    const int quad = warp & 3;
    const int half = e >> 2;
    int acc = 0, round = 0;
    uint32_t acc_phase = 0;
    TileRec rec = tile_seq_get(recs, kSeqCap, tm, a.geom, 0, blockIdx.x, gridDim.x);
    while (rec.row0 >= 0) {
      ++round;
      const int r = quad * 32 + lane;
      int64_t out_row = -1;
      if (r < rec.rows) {
        if (a.out_cyclic_rows) {
          const int i = (rec.pair & 0xFFFF) / q;
          out_row = (int64_t)(rec.row0 + r - i * a.out_cyclic_rows) * q + i;
        } else {
          out_row = a.perm ? __ldg(a.perm + rec.row0 + r) : (rec.row0 + r);
        }
      }
      bool ok = wait_bar(smem_u32(&ctl->tmem_full[acc]), acc_phase, ctl, a.status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      if (e == 0 && lane == 0) ALG_TRACE(2, 1);
      tc_fence_after();
      const uint32_t taddr =
          tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * C::kAccStride + half * C::kHalf);
      const int col_base = rec.n0 + half * C::kHalf;
#pragma unroll 1
      for (int c0 = 0; c0 < C::kHalf; c0 += 32) {
        uint32_t v[32];
        tc_ld_32x32(taddr + (uint32_t)c0, v);
        tc_wait_ld();
        if (out_row >= 0) {
          float f[32];
#pragma unroll
          for (int x = 0; x < 32; ++x) f[x] = __uint_as_float(v[x]);
          finish_and_store_32(f, a, out_row, col_base + c0);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&ctl->tmem_empty[acc]));
      if (e == 0 && lane == 0) ALG_TRACE(2, 2);
      if (++acc == 2) acc = 0, acc_phase ^= 1u;
      rec = tile_seq_get(recs, kSeqCap, tm, a.geom, round, blockIdx.x, gridDim.x);
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
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)C::kTmemCols)
                 : "memory");
  }
}

PFN_cuTensorMapEncodeTiled_v12000 g_encode = nullptr;

template <int TILE_N>
cudaError_t launch_t(const ProjArgs &a, int num_sms, cudaStream_t st) {
  using C = Cfg<TILE_N>;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(proj_tc_kernel<TILE_N>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  const int smem_bytes = C::kFixedSmemBytes + (int)tile_map_bytes(a.n_classes);
  if (smem_bytes > 227 * 1024) return cudaErrorInvalidConfiguration;
  CUtensorMap tmA, tmB;
  cudaError_t e = make_map_a(&tmA, a);
  if (e != cudaSuccess) return e;
  ProjArgs b = a;
  b.b_3d = make_map_b3d(&tmB, a, TILE_N / 64) == cudaSuccess;
  if (!b.b_3d) {
    e = make_map_2d(&tmB, a.W, (uint64_t)a.N, (uint64_t)a.K, (uint64_t)a.ldw * 2, 64, kTcBlockK);
    if (e != cudaSuccess) return e;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(num_sms, 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = std::getenv("ALGPROJ_NO_PDL") ? 0 : 1;
  e = cudaLaunchKernelEx(&cfg, proj_tc_kernel<TILE_N>, tmA, tmB, b);
  count_launch(1);
  return e;
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
  if (a.N % 64 || std::getenv("ALGPROJ_B2D")) return cudaErrorInvalidValue;
  cuuint64_t dims[3] = {64, (cuuint64_t)a.K, (cuuint64_t)(a.N / 64)};
  cuuint64_t strides[2] = {(cuuint64_t)a.ldw * 2, 128};
  cuuint32_t box[3] = {64, kTcBlockK, (cuuint32_t)chunks};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(a.W), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

cudaError_t make_map_a(CUtensorMap *map, const ProjArgs &a) {
  if (!a.a_cyclic_rows)
    return make_map_2d(map, a.X, (uint64_t)a.K, (uint64_t)a.M, (uint64_t)a.ldx * 2, kTcBlockK, kTcTileM);
  cuuint64_t dims[3] = {(cuuint64_t)a.K, (cuuint64_t)a.q, (cuuint64_t)a.a_cyclic_rows};
  cuuint64_t strides[2] = {(cuuint64_t)a.ldx * 2, (cuuint64_t)a.ldx * 2 * (cuuint64_t)a.q};
  cuuint32_t box[3] = {kTcBlockK, 1, kTcTileM};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(a.X), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
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

cudaError_t launch_proj_tc(const ProjArgs &a, int tile_n, int num_sms, cudaStream_t st) {
  cudaError_t e = tc_init();
  if (e != cudaSuccess) return e;
  if (tile_n == 256) return launch_t<256>(a, num_sms, st);
  if (tile_n == 192) return launch_t<192>(a, num_sms, st);
  if (tile_n == 128) return launch_t<128>(a, num_sms, st);
  return cudaErrorInvalidValue;
}

}  // namespace algproj
