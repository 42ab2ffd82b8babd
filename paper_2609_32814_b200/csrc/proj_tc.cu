// Grouped bf16 GEMM over the interaction table for sm_100a: TMA-fed shared-memory tiles,
// tcgen05.mma with the accumulator in tensor memory, persistent CTAs pulling output tiles from
// a device-built list through an atomic counter.
//
// One output tile = 128 rows of one row type i  x  TILE_N columns of one output group j.  All
// kept products of that block (x_k W_kj for k in B(i,j); Eq. recursive-row-action -- for the
// Q_q law x_i W_ij + x_j W_jj, Eqs. typed-diag/off) are issued back to back into the SAME
// TMEM accumulator, so no partial sum ever reaches HBM ("one forward kernel accumulates both
// endpoint products before writing the output", Section "Kernels").
//
// Operands: A = type-bucketed rows, K-contiguous (K-major), 128B-swizzled 128x64 tiles.
//           B = the canonical K x N bank, N-contiguous (MN-major), 64(k) x 64(n) swizzled boxes.
// Warp roles (192 threads): warp 0 = tile scheduler + TMA producer (one lane), warp 1 = TMEM
// allocator + MMA issuer (one lane), warps 2..5 = epilogue (TMEM -> registers -> bias /
// activation -> row scatter to global).  The accumulator is double buffered in TMEM so the
// epilogue of tile t overlaps the main loop of tile t+1.
//
// Every wait on an mbarrier is bounded: on expiry the CTA raises ALG_ERR_DEVICE_TIMEOUT in the
// handle's status word, all roles leave their loops, TMEM is released and the kernel returns.
#include <cuda.h>
#include <cudaTypedefs.h>

#include "common.cuh"

namespace algproj {

namespace {

constexpr int kRing = 4;                       // scheduler ring slots
constexpr long long kTimeoutCycles = 4000000000LL;  // ~2 s at B200 clocks

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
      "l"(map), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tc_ld_32x32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor (sm_100 format): start address, leading / stride byte
// offsets (all >> 4), descriptor version 1, 128-byte swizzle.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= 1ull << 46;
  d |= 2ull << 61;
  return d;
}

__device__ __forceinline__ float gelu_erf(float z) { return 0.5f * z * (1.0f + erff(z * 0.70710678118654752f)); }
__device__ __forceinline__ float gelu_tanh(float z) {
  float u = 0.7978845608028654f * (z + 0.044715f * z * z * z);
  return 0.5f * z * (1.0f + tanhf(u));
}

struct Ctl {
  uint64_t full[8];
  uint64_t empty[8];
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint64_t sched_full[kRing];
  uint64_t sched_empty[kRing];
  TileRec ring[kRing];
  uint32_t tmem_base;
  volatile int abort_flag;
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

template <int TILE_N>
struct Cfg {
  static constexpr int kStages = (TILE_N == 256) ? 4 : 6;
  static constexpr int kABytes = kTcTileM * kTcBlockK * 2;      // 16 KB
  static constexpr int kBChunkBytes = kTcBlockK * 64 * 2;       // one 64(k) x 64(n) box: 8 KB
  static constexpr int kBBytes = kBChunkBytes * (TILE_N / 64);
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kTmemCols = 2 * TILE_N;                   // two accumulators
  static constexpr int kSmemBytes = kStages * kStageBytes + (int)sizeof(Ctl) + 1024;
  // instruction descriptor: D=f32, A=B=bf16, A K-major, B MN-major, N, M=128
  static constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | (1u << 16) |
                                     ((uint32_t)(TILE_N >> 3) << 17) | ((uint32_t)(kTcTileM >> 4) << 24);
};

template <int TILE_N>
__global__ void __launch_bounds__(192, 1)
proj_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const ProjArgs a) {
  using C = Cfg<TILE_N>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  Ctl *ctl = (Ctl *)(smem + C::kStages * C::kStageBytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const DevTable *__restrict__ tab = a.tab;
  const int q = tab->q;

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::kStages; ++s) {
      mbar_init(smem_u32(&ctl->full[s]), 1);
      mbar_init(smem_u32(&ctl->empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&ctl->tmem_full[b]), 1);
      mbar_init(smem_u32(&ctl->tmem_empty[b]), 4);
    }
    for (int s = 0; s < kRing; ++s) {
      mbar_init(smem_u32(&ctl->sched_full[s]), 1);
      mbar_init(smem_u32(&ctl->sched_empty[s]), 5);
    }
    ctl->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmA) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmB) : "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)),
                 "r"((uint32_t)C::kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;

  if (warp == 0) {
    // ---------------- scheduler + TMA producer (one lane) ----------------
    if (lane == 0) {
      const int n_tiles = a.hdr->n_tiles[a.list];
      int *counter = const_cast<int *>(&a.hdr->counter[a.list]);
      int stage = 0, slot = 0;
      uint32_t phase = 0, sphase = 0;
      bool ok = true;
      while (ok) {
        ok = wait_bar(smem_u32(&ctl->sched_empty[slot]), sphase ^ 1u, ctl, a.status);
        if (!ok) break;
        const int t = atomicAdd(counter, 1);
        TileRec rec;
        if (t < n_tiles) rec = a.tiles[t];
        else rec.row0 = -1, rec.rows = 0, rec.pair = 0, rec.n0 = 0;
        ctl->ring[slot] = rec;
        mbar_arrive(smem_u32(&ctl->sched_full[slot]));
        if (++slot == kRing) slot = 0, sphase ^= 1u;
        if (rec.row0 < 0) break;
        const uint32_t mask = tab->keep[rec.pair];
        for (int k = 0; k < q && ok; ++k) {
          if (!((mask >> k) & 1u)) continue;
          const int k_end = tab->so[k + 1];
          for (int k0 = tab->so[k]; k0 < k_end; k0 += kTcBlockK) {
            ok = wait_bar(smem_u32(&ctl->empty[stage]), phase ^ 1u, ctl, a.status);
            if (!ok) break;
            const uint32_t bar = smem_u32(&ctl->full[stage]);
            const uint32_t sa = smem_u32(smem + stage * C::kStageBytes);
            mbar_expect_tx(bar, (uint32_t)C::kStageBytes);
            tma_load_2d(sa, &tmA, bar, k0, rec.row0);
#pragma unroll
            for (int c = 0; c < TILE_N / 64; ++c)
              tma_load_2d(sa + C::kABytes + c * C::kBChunkBytes, &tmB, bar, rec.n0 + c * 64, k0);
            if (++stage == C::kStages) stage = 0, phase ^= 1u;
          }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer (one lane) ----------------
    if (lane == 0) {
      int stage = 0, slot = 0, acc = 0;
      uint32_t phase = 0, sphase = 0, acc_phase = 0;
      bool ok = true;
      while (ok) {
        ok = wait_bar(smem_u32(&ctl->sched_full[slot]), sphase, ctl, a.status);
        if (!ok) break;
        const TileRec rec = ctl->ring[slot];
        mbar_arrive(smem_u32(&ctl->sched_empty[slot]));
        if (++slot == kRing) slot = 0, sphase ^= 1u;
        if (rec.row0 < 0) break;
        ok = wait_bar(smem_u32(&ctl->tmem_empty[acc]), acc_phase ^ 1u, ctl, a.status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * TILE_N);
        const uint32_t mask = tab->keep[rec.pair];
        uint32_t accumulate = 0;
        for (int k = 0; k < q && ok; ++k) {
          if (!((mask >> k) & 1u)) continue;
          const int n_kb = (tab->so[k + 1] - tab->so[k]) / kTcBlockK;
          for (int kb = 0; kb < n_kb; ++kb) {
            ok = wait_bar(smem_u32(&ctl->full[stage]), phase, ctl, a.status);
            if (!ok) break;
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
        if (++acc == 2) acc = 0, acc_phase ^= 1u;
      }
    }
  } else {
    // ---------------- epilogue warps: TMEM lanes [32*(warp%4), +32) ----------------
    const int quad = warp & 3;
    int slot = 0, acc = 0;
    uint32_t sphase = 0, acc_phase = 0;
    const bool y_bf16 = a.y_bf16 != 0;
    while (true) {
      bool ok = wait_bar(smem_u32(&ctl->sched_full[slot]), sphase, ctl, a.status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      const TileRec rec = ctl->ring[slot];
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&ctl->sched_empty[slot]));
      if (++slot == kRing) slot = 0, sphase ^= 1u;
      if (rec.row0 < 0) break;
      ok = wait_bar(smem_u32(&ctl->tmem_full[acc]), acc_phase, ctl, a.status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const int r = quad * 32 + lane;
      int64_t out_row = -1;
      if (r < rec.rows) out_row = a.perm ? a.perm[rec.row0 + r] : (rec.row0 + r);
      const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * TILE_N);
#pragma unroll 1
      for (int c0 = 0; c0 < TILE_N; c0 += 32) {
        uint32_t v[32];
        tc_ld_32x32(taddr + (uint32_t)c0, v);
        tc_wait_ld();
        if (out_row >= 0) {
          const int col = rec.n0 + c0;
          float f[32];
#pragma unroll
          for (int e = 0; e < 32; ++e) f[e] = __uint_as_float(v[e]);
          if (a.bias) {
            const __nv_bfloat16 *b = (const __nv_bfloat16 *)a.bias + col;
#pragma unroll
            for (int e = 0; e < 32; ++e) f[e] += __bfloat162float(__ldg(b + e));
          }
          if (a.act == ALG_ACT_GELU_ERF) {
#pragma unroll
            for (int e = 0; e < 32; ++e) f[e] = gelu_erf(f[e]);
          } else if (a.act == ALG_ACT_GELU_TANH) {
#pragma unroll
            for (int e = 0; e < 32; ++e) f[e] = gelu_tanh(f[e]);
          }
          if (y_bf16) {
            uint4 *dst = (uint4 *)((__nv_bfloat16 *)a.Y + out_row * a.ldy + col);
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              uint32_t w[4];
#pragma unroll
              for (int h = 0; h < 4; ++h) {
                __nv_bfloat162 p = __floats2bfloat162_rn(f[g * 8 + 2 * h], f[g * 8 + 2 * h + 1]);
                w[h] = *(uint32_t *)&p;
              }
              dst[g] = make_uint4(w[0], w[1], w[2], w[3]);
            }
          } else {
            float4 *dst = (float4 *)((float *)a.Y + out_row * a.ldy + col);
#pragma unroll
            for (int g = 0; g < 8; ++g) dst[g] = make_float4(f[g * 4], f[g * 4 + 1], f[g * 4 + 2], f[g * 4 + 3]);
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&ctl->tmem_empty[acc]));
      if (++acc == 2) acc = 0, acc_phase ^= 1u;
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

template <int TILE_N>
cudaError_t launch_t(const ProjArgs &a, int num_sms, cudaStream_t st) {
  using C = Cfg<TILE_N>;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(proj_tc_kernel<TILE_N>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  CUtensorMap tmA, tmB;
  cudaError_t e = make_map_2d(&tmA, a.X, (uint64_t)a.K, (uint64_t)a.M, (uint64_t)a.ldx * 2, kTcBlockK, kTcTileM);
  if (e != cudaSuccess) return e;
  e = make_map_2d(&tmB, a.W, (uint64_t)a.N, (uint64_t)a.K, (uint64_t)a.ldw * 2, 64, kTcBlockK);
  if (e != cudaSuccess) return e;
  proj_tc_kernel<TILE_N><<<num_sms, 192, C::kSmemBytes, st>>>(tmA, tmB, a);
  count_launch(1);
  return cudaGetLastError();
}

}  // namespace

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
  if (tile_n == 128) return launch_t<128>(a, num_sms, st);
  return cudaErrorInvalidValue;
}

}  // namespace algproj
