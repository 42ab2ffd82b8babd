// Grouped bf16 GEMM over the interaction table with CTA pairs (tcgen05 cta_group::2).
//
// Two CTAs of a cluster share one 256-row x N-column output tile (N = 256, or the 128-column rest
// of an output group): CTA r owns rows [128 r, 128 r + 128) of the tile and their accumulator in
// its own tensor memory, loads its own 128 x 64 A block and HALF of the 64 x N B block per
// K step, and the leader CTA's single MMA thread issues tcgen05.mma.cta_group::2 (M = 256), which
// reads A and the B halves from both CTAs' shared memory.  Compared with one-CTA 128 x 256
// tiles this cuts the bytes fetched per FLOP by a third (32 KB instead of 48 KB per 128x256x64
// block of work), which is what the ~1.2 us load latency of a busy L2 needs: six stages then
// cover 3072 tensor-pipe cycles of look-ahead instead of 2048.
//
// As in the one-CTA kernel all kept products of a block (x_k W_kj, k in B(i,j);
// Eq. recursive-row-action) accumulate in one TMEM tile, the accumulator is double buffered, and
// the epilogue (8 warps per CTA) applies bias / GELU and scatters rows to their original order.
//
// Synchronisation across the pair:
//   full[s]       lives in the leader; both CTAs' TMA loads complete on it (2-SM load form).
//   empty[s]      one per CTA, both released by one multicast tcgen05.commit of the leader.
//   tmem_full[b]  one per CTA, multicast commit after the last MMA of a tile.
//   tmem_empty[b] lives in the leader; all 16 epilogue warps of the pair arrive on it.
// Every wait is bounded; on expiry the CTA sets ALG_ERR_DEVICE_TIMEOUT, leaves its loops, meets
// its peer at the final cluster barrier, frees its tensor memory and returns.
#include "tc_common.cuh"

namespace algproj {

using namespace tc;

ALG_TRACE_DEFINE(proj_tc2)

namespace {

constexpr int kEpiWarps = 8;
constexpr int kProducerWarpB = 2 + kEpiWarps;   // second TMA producer, after the epilogue warps
constexpr int kThreads = 32 * (3 + kEpiWarps);
constexpr int kMaxStages = 7;
constexpr int kSeqCap = kTc2SeqCap;   // precomputed tile records per CTA pair
constexpr int kABytes = 128 * kTcBlockK * 2;              // 16 KB: this CTA's rows
constexpr int kBChunkBytes = kTcBlockK * 64 * 2;           // one 64(k) x 64(n) box
constexpr int kBMaxBytes = kBChunkBytes * (kTc2TileN / 128);  // this CTA's half of the B block: 16 KB
constexpr int kStageBytes = kABytes + kBMaxBytes;          // 32 KB
constexpr int kAccStride = kTc2TileN;                      // TMEM columns per accumulator
constexpr int kTmemCols = 2 * kAccStride;                  // 512
constexpr uint32_t kPeerMask = 0xFEFFFFFFu;                // shared::cluster address -> the even CTA of the pair

struct Ctl2 {
  uint64_t full[kMaxStages];
  uint64_t empty[kMaxStages];
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint32_t tmem_base;
  volatile int abort_flag;
  long long wait_limit;     // bound of every wait, in clock64 cycles
  int so[kMaxQ + 1];
  uint32_t keep[1];  // q*q entries follow, then q*q uint16 K-block counts (the request is sized for them)
};
constexpr int kMaxSmem = 227 * 1024;
inline int smem_bytes(int n_stages, int q, int n_classes) {
  return n_stages * kStageBytes + (int)sizeof(Ctl2) + q * q * 6 + 16 + kSeqCap * 16 + (int)tile_map_bytes(n_classes) + 32 +
         1024;
}
inline int pick_stages(int q, int n_classes) {
  return smem_bytes(kMaxStages, q, n_classes) <= kMaxSmem ? kMaxStages : kMaxStages - 1;
}

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_remote(uint32_t local_bar, uint32_t target_rank) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_bar), "r"(target_rank));
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote) : "memory");
}
// 2-SM form of the tiled TMA load: data lands in this CTA's shared memory, completion is
// signalled on the leader CTA's barrier.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, uint32_t leader_bar, int c0,
                                                 int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(
          dst),
      "l"(map), "r"(leader_bar), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap *map, uint32_t leader_bar, int c0,
                                                 int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];" ::"r"(
          dst),
      "l"(map), "r"(leader_bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ void tc2_commit_both(uint32_t bar) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
      "h"((uint16_t)3)
      : "memory");
}
__device__ __forceinline__ void tc2_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                             uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}

__device__ __noinline__ bool wait_slow2(uint32_t bar, uint32_t parity, Ctl2 *ctl, int *status) {
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
__device__ __forceinline__ bool wait_bar2(uint32_t bar, uint32_t parity, Ctl2 *ctl, int *status) {
  if (mbar_try_wait(bar, parity)) return true;
  return wait_slow2(bar, parity, ctl, status);
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
proj_tc2_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const ProjArgs a,
                const int n_stages) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const int tab_q = a.q;
  Ctl2 *ctl = (Ctl2 *)(smem + n_stages * kStageBytes);
  uint16_t *nkb = (uint16_t *)(ctl->keep + tab_q * tab_q);
  TileRec *recs = (TileRec *)(((uintptr_t)(nkb + tab_q * tab_q) + 15) & ~(uintptr_t)15);
  TileMap *tm = (TileMap *)(recs + kSeqCap);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const DevTable *__restrict__ tab = a.tab;
  const int q = tab_q;
  const uint32_t rank = cluster_ctarank();          // 0 = leader
  ALG_TRACE_VARS;
  ALG_TRACE_CTA(0, a.act ? 0 : 1);

  if (threadIdx.x == 0) {
    for (int s = 0; s < n_stages; ++s) {
      mbar_init(smem_u32(&ctl->full[s]), 1);
      mbar_init(smem_u32(&ctl->empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&ctl->tmem_full[b]), 1);
      mbar_init(smem_u32(&ctl->tmem_empty[b]), 2 * kEpiWarps);
    }
    ctl->abort_flag = 0;
    ctl->wait_limit = a.wait_limit;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmA) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmB) : "memory");
  }
  for (int e = threadIdx.x; e < q * q; e += kThreads) ctl->keep[e] = a.st.valid ? a.st.keep[e] : tab->keep[e];
  for (int e = threadIdx.x; e <= q; e += kThreads) ctl->so[e] = a.st.valid ? a.st.so[e] : tab->so[e];
  for (int e = threadIdx.x; e < q * q; e += kThreads) {
    const uint32_t mask = a.st.valid ? a.st.keep[e] : tab->keep[e];
    int n = 0;
    for (int k = 0; k < q; ++k)
      if ((mask >> k) & 1u) n += (a.st.valid ? a.st.so[k + 1] - a.st.so[k] : tab->so[k + 1] - tab->so[k]) / kTcBlockK;
    nkb[e] = (uint16_t)n;
  }
  if (warp == 1) {  // both CTAs of the pair allocate together, same shared-memory slot
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)),
                 "r"((uint32_t)kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  // Programmatic dependent launch: everything above touches only this CTA's own state.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  tile_map_build(tm, tab, a.st, a.q, a.n_classes, a.offsets, a.cyclic_rows, a.M, a.geom);
  tile_seq_build(recs, kSeqCap, tm, a.geom, blockIdx.x >> 1, gridDim.x >> 1, nkb);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // the peer's barriers are initialised before anything signals them
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;

  // Producer and MMA roles run warp-uniformly (all lanes execute loops and waits, one elected lane
  // issues), so that the operands of the copy / MMA / commit instructions stay in uniform
  // registers; loop bounds read from shared memory are broadcast with a shuffle.
  if (warp == 0 || warp == kProducerWarpB) {
    // ---------------- TMA producers (both CTAs): warp 0 loads A, the last warp loads the B half ------
    const bool loads_a = warp == 0;
    int stage = 0, round = 0;
    uint32_t phase = 0;
    bool ok = true;
    const uint32_t full0 = smem_u32(&ctl->full[0]), empty0 = smem_u32(&ctl->empty[0]);
    const uint32_t smem0 = smem_u32(smem);
    TileRec rec = tile_seq_get(recs, tm, a.geom, 0, blockIdx.x >> 1, gridDim.x >> 1, nkb);
    while (ok && __shfl_sync(0xffffffffu, rec.row0, 0) >= 0) {
      ++round;
      if (loads_a && lane == 0) ALG_TRACE(0, 1);
      const int pair = __shfl_sync(0xffffffffu, rec.pair & 0xFFFF, 0);
      const int cols = __shfl_sync(0xffffffffu, rec.pair >> 16, 0);
      const int row0 = __shfl_sync(0xffffffffu, rec.row0, 0);
      const int n0 = __shfl_sync(0xffffffffu, rec.n0, 0);
      const uint32_t mask = __shfl_sync(0xffffffffu, ctl->keep[pair], 0);
      const int half_cols = cols >> 1;                       // B columns this CTA loads: 128 or 64
      const int n_chunks = half_cols >> 6;
      const uint32_t tx_bytes = 2u * (uint32_t)(kABytes + n_chunks * kBChunkBytes);
      const int type_i = pair / q;
      const int row = row0 + 128 * (int)rank - (a.a_cyclic_rows ? type_i * a.a_cyclic_rows : 0);
      const int col = n0 + (int)rank * half_cols;
      for (int k = 0; k < q && ok; ++k) {
        if (!((mask >> k) & 1u)) continue;
        const int k_begin = __shfl_sync(0xffffffffu, ctl->so[k], 0);
        const int k_end = __shfl_sync(0xffffffffu, ctl->so[k + 1], 0);
        for (int k0 = k_begin; k0 < k_end; k0 += kTcBlockK) {
          ok = __all_sync(0xffffffffu, wait_bar2(empty0 + 8u * (uint32_t)stage, phase ^ 1u, ctl, a.status));
          if (!ok) break;
          const uint32_t own_bar = full0 + 8u * (uint32_t)stage;
          const uint32_t sa = smem0 + (uint32_t)stage * (uint32_t)kStageBytes;
          const uint32_t bar = own_bar & kPeerMask;
          if (elect_one()) {
            if (loads_a) {
              if (rank == 0) mbar_expect_tx(own_bar, tx_bytes);
              if (a.a_cyclic_rows) tma_load_3d_pair(sa, &tmA, bar, k0, type_i, row);
              else tma_load_2d_pair(sa, &tmA, bar, k0, row);
            } else {
              for (int c = 0; c < n_chunks; ++c)
                tma_load_2d_pair(sa + kABytes + c * kBChunkBytes, &tmB, bar, col + c * 64, k0);
            }
          }
          __syncwarp();
          if (++stage == n_stages) stage = 0, phase ^= 1u;
        }
      }
      if (loads_a && lane == 0) ALG_TRACE(0, 2);
      rec = tile_seq_get(recs, tm, a.geom, round, blockIdx.x >> 1, gridDim.x >> 1, nkb);
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer (leader CTA) ----------------
    if (rank == 0) {
      int stage = 0, acc = 0, round = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      const uint32_t full0 = smem_u32(&ctl->full[0]), empty0 = smem_u32(&ctl->empty[0]);
      const uint32_t tfull0 = smem_u32(&ctl->tmem_full[0]), tempty0 = smem_u32(&ctl->tmem_empty[0]);
      const uint64_t da0 = make_smem_desc(smem_u32(smem), 16, 1024);
      const uint64_t db0 = make_smem_desc(smem_u32(smem) + kABytes, kBChunkBytes, 1024);
      TileRec rec = tile_seq_get(recs, tm, a.geom, 0, blockIdx.x >> 1, gridDim.x >> 1, nkb);
      while (ok && __shfl_sync(0xffffffffu, rec.row0, 0) >= 0) {
        ++round;
        if (lane == 0) ALG_TRACE(1, 1);
        const int n_kb = __shfl_sync(0xffffffffu, (int)((uint32_t)rec.rows >> 16), 0);
        const int cols = __shfl_sync(0xffffffffu, rec.pair >> 16, 0);
        ok = __all_sync(0xffffffffu, wait_bar2(tempty0 + 8u * (uint32_t)acc, acc_phase ^ 1u, ctl, a.status));
        if (!ok) break;
        if (lane == 0) ALG_TRACE(1, 2);
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * kAccStride);
        // instruction descriptor: D=f32, A=B=bf16, A K-major, B MN-major, N = cols, M = 256
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | (1u << 16) |
                               ((uint32_t)(cols >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
        for (int kb = 0; kb < n_kb; ++kb) {
          ok = __all_sync(0xffffffffu, wait_bar2(full0 + 8u * (uint32_t)stage, phase, ctl, a.status));
          if (!ok) break;
          if (kb == 0 && lane == 0) ALG_TRACE(1, 3);
          tc_fence_after();
          const uint64_t da = da0 + (uint64_t)((uint32_t)stage * (uint32_t)(kStageBytes >> 4));
          const uint64_t db = db0 + (uint64_t)((uint32_t)stage * (uint32_t)(kStageBytes >> 4));
          if (elect_one()) {
            tc2_mma_bf16(d_tmem, da, db, idesc, kb ? 1u : 0u);
#pragma unroll
            for (int kk = 1; kk < kTcBlockK / 16; ++kk)
              tc2_mma_bf16(d_tmem, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 128), idesc, 1u);
            tc2_commit_both(empty0 + 8u * (uint32_t)stage);
          }
          __syncwarp();
          if (++stage == n_stages) stage = 0, phase ^= 1u;
        }
        if (!ok) break;
        if (elect_one()) tc2_commit_both(tfull0 + 8u * (uint32_t)acc);
        __syncwarp();
        if (lane == 0) ALG_TRACE(1, 4);
        if (++acc == 2) acc = 0, acc_phase ^= 1u;
        rec = tile_seq_get(recs, tm, a.geom, round, blockIdx.x >> 1, gridDim.x >> 1, nkb);
      }
    }
  } else {
    // ---------------- epilogue: warp e handles TMEM lanes [32*(warp%4), +32), column half e/4 ----
    const int e = warp - 2;
    const int quad = warp & 3;
    const int half = e >> 2;
    int acc = 0, round = 0;
    uint32_t acc_phase = 0;
    TileRec rec = tile_seq_get(recs, tm, a.geom, 0, blockIdx.x >> 1, gridDim.x >> 1, nkb);
    while (rec.row0 >= 0) {
      ++round;
      const int cols = rec.pair >> 16;
      const int half_cols = cols >> 1;
      const int r = 128 * (int)rank + quad * 32 + lane;   // row inside the 256-row tile
      int64_t out_row = -1;
      if (r < (rec.rows & 0xFFFF)) {
        if (a.out_cyclic_rows) {
          const int i = (rec.pair & 0xFFFF) / q;
          out_row = (int64_t)(rec.row0 + r - i * a.out_cyclic_rows) * q + i;
        } else {
          out_row = a.perm ? __ldg(a.perm + rec.row0 + r) : (rec.row0 + r);
        }
        if (out_row >= a.M) out_row = -1;   // never store outside Y, whatever the tile record says
      }
      bool ok = wait_bar2(smem_u32(&ctl->tmem_full[acc]), acc_phase, ctl, a.status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      if (e == 0 && lane == 0) ALG_TRACE(2, 1);
      tc_fence_after();
      const uint32_t taddr =
          tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * kAccStride + half * half_cols);
      const int col_base = rec.n0 + half * half_cols;
#pragma unroll 1
      for (int c0 = 0; c0 < half_cols; c0 += 32) {
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
      if (lane == 0) {
        if (rank == 0) mbar_arrive(smem_u32(&ctl->tmem_empty[acc]));
        else mbar_arrive_remote(smem_u32(&ctl->tmem_empty[acc]), 0);
      }
      if (e == 0 && lane == 0) ALG_TRACE(2, 2);
      if (++acc == 2) acc = 0, acc_phase ^= 1u;
      rec = tile_seq_get(recs, tm, a.geom, round, blockIdx.x >> 1, gridDim.x >> 1, nkb);
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
  cluster_sync_all();  // neither CTA leaves while its peer may still signal or read its shared memory
  ALG_TRACE_CTA(1, a.act ? 0 : 1);
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kTmemCols)
                 : "memory");
  }
}

}  // namespace

int tc2_max_pairs(int num_sms) {
  static int max_pairs = -1;
  if (max_pairs >= 0) return max_pairs;
  if (cudaFuncSetAttribute(proj_tc2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem) != cudaSuccess)
    return 0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * (num_sms / 2));
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem_bytes(kMaxStages - 1, kMaxQ, kMaxClasses);
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, proj_tc2_kernel, &cfg) != cudaSuccess || n < 1) return 0;
  max_pairs = n < num_sms / 2 ? n : num_sms / 2;
  if (max_pairs > kMaxWorkers) max_pairs = kMaxWorkers;
  return max_pairs;
}

cudaError_t launch_proj_tc2(const ProjArgs &a, int num_sms, cudaStream_t st) {
  cudaError_t e = tc_init();
  if (e != cudaSuccess) return e;
  const int pairs = tc2_max_pairs(num_sms);
  if (pairs < 1) return cudaErrorInvalidConfiguration;
  const int q = a.q;
  const int n_stages = pick_stages(q, a.n_classes);
  if (smem_bytes(n_stages, q, a.n_classes) > kMaxSmem) return cudaErrorInvalidConfiguration;
  CUtensorMap tmA, tmB;
  e = make_map_a(&tmA, a);
  if (e != cudaSuccess) return e;
  e = make_map_2d(&tmB, a.W, (uint64_t)a.N, (uint64_t)a.K, (uint64_t)a.ldw * 2, 64, kTcBlockK);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs, 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = smem_bytes(n_stages, q, a.n_classes);
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  e = cudaLaunchKernelEx(&cfg, proj_tc2_kernel, tmA, tmB, a, n_stages);
  count_launch(1);
  return e;
}

}  // namespace algproj
