// Decode step of the whole two-map FFN in ONE launch:  Y = act(X *_q W_up + b_up) *_q W_down + b_down
// for M <= 16 new rows (Section "One-Token Inference": one new row per sequence, typed by its
// absolute position; the regime is bound by weight traffic and by latency, not by arithmetic).
//
// Why one launch.  A 768 -> 3072 -> 768 layer streams 9.4 MB of weights, 1.4 us of HBM time, while a
// chain of dependent kernels pays several microseconds of serial latency per kernel.  Here every
// CTA requests its slice of BOTH banks the moment it starts -- before it waits for the previous
// kernel of the stream (programmatic dependent launch) -- and a CTA needs less than half of an SM's
// shared memory, so the CTAs of the next layer's launch sit beside the ones of the running layer
// and their weight stream overlaps its arithmetic.
//
// Decomposition.  No reduction across CTAs anywhere: CTA c owns `su` columns of the hidden state
// (all D input rows of W_up for them) and `sd` columns of the output (all F rows of W_down).
//   before the wait : row types read speculatively -> input groups some row needs (blocks W_kj that
//                     no present row type uses are never fetched) -> both slices requested with
//                     16-byte asynchronous copies (a slice is only 16-48 bytes wide per weight row;
//                     tiled TMA boxes that narrow were measured no faster), each asking L2 for the
//                     whole 128-byte line the neighbouring CTAs need too.
//   after the wait  : X staged in shared memory (all groups, unmasked) while the row types are read
//                     again; if they differ, the blocks that are missing are requested now.
//   up phase        : 8 warps split the K steps; mma.sync m16n8k16 (bf16 x bf16 -> fp32); the rule
//                     "row b uses block k only if k in B(t_b, j)" is applied by clearing the A
//                     fragment rows that do not use the block; the 8 partial tiles are summed in a
//                     fixed order through shared memory; bias, activation, bf16 -> H in global memory.
//   exchange        : producers publish with fence + one atomic add on a counter; consumers poll it
//                     (bounded), the last consumer clears the counters for the next launch.
//   down phase      : H staged from L2 over the shared memory the W_up slice no longer needs; same
//                     MMA / reduction; bias; Y stored.
// Every wait (mbarriers the copies arrive on, one counter) is bounded by the handle's wait limit; on expiry the CTA
// raises ALG_ERR_DEVICE_TIMEOUT, skips its arithmetic, gives copies in flight time to land and
// returns.
#include <algorithm>

#include "tc_common.cuh"

namespace algproj {

using namespace tc;

ALG_TRACE_DEFINE(ffn_decode)

namespace {

constexpr int kThreads = 256, kWarps = 8;
constexpr int kSmemBudget = 112 * 1024;   // two CTAs (this launch and the next layer's) per SM

constexpr int kLoaders = 64;    // threads per weight slice: warps 0-1 fetch W_up, warps 2-3 fetch W_down
constexpr int kStagers = 128;   // warps 4-7 stage the activations

struct Ctl {
  uint64_t bar_up, bar_dn, bar_miss, bar_x;
  int so_d[kMaxQ + 1], so_f[kMaxQ + 1];   // input-group offsets of the up (D) / down (F) projection
  uint32_t need_up, need_dn;              // input groups some present row needs for this CTA's strips
  uint32_t miss_up, miss_dn;              // needed by the final types, not requested for the speculative ones
  uint32_t rows_up[kMaxQ], rows_dn[kMaxQ];  // bit m: row m uses input group k
  uint32_t bad_rows;
  volatile int abort_flag;
  volatile int go;
};

__device__ __forceinline__ void cp_async_16_zfill(uint32_t dst, const void *src, bool valid) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(valid ? 16 : 0) : "memory");
}
__device__ __forceinline__ void cp_async_16_l2line(uint32_t dst, const void *src) {
  asm volatile("cp.async.cg.shared.global.L2::128B [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
// arrives on the barrier once every copy this thread has issued so far has landed
__device__ __forceinline__ void cp_async_arrive(uint32_t bar) {
  asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x2(uint32_t addr, uint32_t &r0, uint32_t &r1) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x2_trans(uint32_t addr, uint32_t &r0, uint32_t &r1) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0,%1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned *p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ float act_f(float z, int act) {
  if (act == ALG_ACT_GELU_ERF) return 0.5f * z * (1.0f + erff(z * 0.70710678118654752f));
  if (act == ALG_ACT_GELU_TANH) {
    float u = 0.7978845608028654f * (z + 0.044715f * z * z * z);
    return 0.5f * z * (1.0f + tanhf(u));
  }
  return z;
}
// staged activations: [m_pad][kc] bf16, 16-byte pieces XOR-swizzled by the row (conflict-free ldmatrix)
__device__ __forceinline__ uint32_t x_off(int m, int chunk, int pitch_bytes) {
  return (uint32_t)(m * pitch_bytes + ((chunk ^ (m & 7)) << 4));
}

// Warp 0: from the types of the M rows (lane m holds the type of row m, -1 = out of range) to the
// input groups this CTA's strips need and, per group, the rows that use it.
__device__ __forceinline__ void derive_masks(Ctl *ctl, const FfnDecodeArgs &a, int my_type, int M, int q, int ju, int jd,
                                             int lane) {
  const bool live = lane < M && my_type >= 0;
  const uint32_t *keep = a.small_q ? a.keep : a.tab_up->keep;   // by value in the kernel parameters when the table is small
  const uint32_t ku = (live && ju >= 0) ? keep[my_type * q + ju] : 0u;
  const uint32_t kd = (live && jd >= 0) ? keep[my_type * q + jd] : 0u;
  const uint32_t nu = __reduce_or_sync(0xffffffffu, ku), nd = __reduce_or_sync(0xffffffffu, kd);
  const uint32_t bad = __ballot_sync(0xffffffffu, lane < M && my_type < 0);
  for (int k = 0; k < q; ++k) {
    const uint32_t vu = __ballot_sync(0xffffffffu, (ku >> k) & 1u), vd = __ballot_sync(0xffffffffu, (kd >> k) & 1u);
    if (lane == 0) ctl->rows_up[k] = vu, ctl->rows_dn[k] = vd;
  }
  if (lane == 0) ctl->need_up = nu, ctl->need_dn = nd, ctl->bad_rows = bad;
}

// What one projection phase (up or down) of a CTA works on.
struct Phase {
  const __nv_bfloat16 *src;   // activations in global memory: X, or H written by the up phase of all CTAs
  int ld, K;                  // their leading dimension; the reduction length (D or F)
  int kc, pitch_bytes;        // staged K chunk and its row pitch
  uint32_t stage_base;        // shared memory of the staged chunk [m_pad][kc], 16-byte pieces XOR-swizzled by row
  uint32_t w_base;            // weight slice [K][cols] in shared memory
  int cols, col0;             // strip width, first column
  const int *so;              // input-group offsets
  const uint32_t *rows_k;     // per input group: rows that use it
  uint32_t need;              // input groups some row needs
  const void *bias;
  int act;
  void *out;                  // H (bf16) or Y
  int out_ld, out_bf16;
  bool first_chunk_staged;    // chunk 0 was requested by the caller already
};
struct Shared {
  Ctl *ctl;
  float *p_sm;
  uint32_t bar_x;
  int M, m_pad, q;
  long long wait_limit;
  int *status;
};

// bounded wait on an mbarrier (all threads)
__device__ __forceinline__ bool wait_bar(const Shared &sh, uint32_t bar, uint32_t parity) {
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (sh.ctl->abort_flag) return false;
    if (clock64() - t0 > sh.wait_limit) {
      sh.ctl->abort_flag = 1;
      atomicExch(sh.status, (int)ALG_ERR_DEVICE_TIMEOUT);
      return false;
    }
  }
  return true;
}

// Warps 4-7 stage one K chunk of an activation matrix (rows >= M are zero) and arrive on bar_x.
__device__ __forceinline__ void stage_chunk(const Shared &sh, const Phase &ph, int kc0, int len) {
  const int tid = threadIdx.x;
  if (tid < kThreads - kStagers) return;
  const bool half_tile = sh.m_pad == 8;
  const int cpr = len >> 3;   // 16-byte pieces per row
  // 128 stagers over m_pad rows: 16 (or 8) neighbouring threads walk along one row
  const int t = tid - (kThreads - kStagers);
  const int tpr = half_tile ? kStagers / 8 : kStagers / 16;
  const int m = half_tile ? (t >> 4) : (t >> 3);
  const bool valid = m < sh.M;
  const __nv_bfloat16 *row = ph.src + (int64_t)(valid ? m : 0) * ph.ld + kc0;
  const uint32_t dst_row = ph.stage_base + (uint32_t)(m * ph.pitch_bytes);
  for (int ch = t & (tpr - 1); ch < cpr; ch += tpr)
    cp_async_16_zfill(dst_row + (uint32_t)((ch ^ (m & 7)) << 4), row + ch * 8, valid);
  cp_async_arrive(sh.bar_x);
}

// One projection phase of a CTA:  out[:, strip] = act(src *_q W[:, strip] + bias).
// The K range is staged chunk by chunk (one chunk for M <= 8 at the benchmark shape).  Warp w takes
// the 16-deep K steps w, w+8, ... of every needed input group, in batches of SETS steps: all
// fragments of a batch are loaded first, then its MMAs go to SETS independent accumulator sets, so
// neither the shared-memory latency nor the chain of dependent MMAs is paid per step.  The rule
// "row b uses block k only if k in B(t_b, j)" is applied by clearing the rows of the A fragment that
// do not use the block.  The 8 warps' partial tiles are then summed in warp order through shared
// memory (deterministic), bias and activation applied, rows < M stored.
// NT = 8-column tiles of the strip.  Returns false when a wait ran out.
template <int NT>
__device__ __forceinline__ bool run_phase_t(const Shared &sh, const Phase &ph, uint32_t &x_parity) {
  constexpr int SETS = NT <= 2 ? 4 : (NT <= 4 ? 2 : 1);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const bool HALF = sh.m_pad == 8;
  const int g = lane >> 2, t4 = lane & 3;
  const int frag_row = (lane & 7) + ((lane >> 3) & 1) * 8;
  const int a_row = HALF ? (lane & 7) : frag_row;
  const int a_sel = HALF ? ((lane >> 3) & 1) : (lane >> 4);
  const uint32_t a_lane = ph.stage_base + (uint32_t)(a_row * ph.pitch_bytes);
  const int a_x = a_row & 7;
  const int w_pitch_bytes = ph.cols * 2;
  const uint32_t w_lane = ph.w_base + (uint32_t)(frag_row * w_pitch_bytes);
  float d[SETS][NT][4];
#pragma unroll
  for (int s = 0; s < SETS; ++s)
#pragma unroll
    for (int o = 0; o < NT; ++o) d[s][o][0] = d[s][o][1] = d[s][o][2] = d[s][o][3] = 0.f;
  bool ok = true;
  for (int kc0 = 0; kc0 < ph.K && ok; kc0 += ph.kc) {
    const int len = min(ph.kc, ph.K - kc0);
    if (kc0 || !ph.first_chunk_staged) {
      if (kc0) __syncthreads();   // the previous chunk has been consumed
      stage_chunk(sh, ph, kc0, len);
    }
    ok = wait_bar(sh, sh.bar_x, x_parity);
    x_parity ^= 1u;
    if (!ok) break;
    for (int k = 0; k < sh.q; ++k) {
      if (!((ph.need >> k) & 1u)) continue;
      const int b = max(ph.so[k], kc0), e = min(ph.so[k + 1], kc0 + len);
      if (b >= e) continue;
      const uint32_t rk = ph.rows_k[k];
      const uint32_t mlo = ((rk >> g) & 1u) ? 0xffffffffu : 0u, mhi = ((rk >> (g + 8)) & 1u) ? 0xffffffffu : 0u;
      for (int kk = b + 16 * warp; kk < e; kk += SETS * 16 * kWarps) {
        uint32_t af[SETS][4], bf[SETS][NT][2];
#pragma unroll
        for (int s = 0; s < SETS; ++s) {
          const int ks = kk + s * 16 * kWarps;
          if (ks < e) {
            const uint32_t a_addr = a_lane + (uint32_t)(((((ks - kc0) >> 3) + a_sel) ^ a_x) << 4);
            if (HALF) {
              ldmatrix_x2(a_addr, af[s][0], af[s][2]);
              af[s][1] = af[s][3] = 0u;
            } else {
              ldmatrix_x4(a_addr, af[s]);
            }
            const uint32_t wrow = w_lane + (uint32_t)(ks * w_pitch_bytes);
#pragma unroll
            for (int o = 0; o < NT; ++o) ldmatrix_x2_trans(wrow + (uint32_t)(o << 4), bf[s][o][0], bf[s][o][1]);
          }
        }
#pragma unroll
        for (int s = 0; s < SETS; ++s) {
          if (kk + s * 16 * kWarps < e) {
            af[s][0] &= mlo, af[s][2] &= mlo, af[s][1] &= mhi, af[s][3] &= mhi;
#pragma unroll
            for (int o = 0; o < NT; ++o) mma_bf16(d[s][o], af[s], bf[s][o][0], bf[s][o][1]);
          }
        }
      }
    }
  }
  __syncthreads();
  if (sh.ctl->abort_flag) return false;
  // ---- the 8 warps' partial tiles -> shared memory -> ordered sum, bias, activation, store ----
  const int cols = ph.cols;
#pragma unroll
  for (int o = 0; o < NT; ++o) {
    float v[4];
#pragma unroll
    for (int x = 0; x < 4; ++x) {
      v[x] = d[0][o][x];
#pragma unroll
      for (int s = 1; s < SETS; ++s) v[x] += d[s][o][x];
    }
    float *p = sh.p_sm + ((warp * sh.m_pad + g) * cols + o * 8 + t4 * 2);
    *(float2 *)p = make_float2(v[0], v[1]);
    if (!HALF) *(float2 *)(p + 8 * cols) = make_float2(v[2], v[3]);
  }
  __syncthreads();
  const int pairs = cols >> 1;
  const int m = tid >> 4;   // 16 rows x 16 threads that walk along the row's column pairs
  for (int pr = tid & 15; pr < pairs && m < sh.M; pr += 16) {
    const int cp = pr * 2;
    float z0 = 0.f, z1 = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
      const float2 v = *(const float2 *)(sh.p_sm + ((w * sh.m_pad + m) * cols + cp));
      z0 += v.x, z1 += v.y;
    }
    const int col = ph.col0 + cp;
    if (ph.bias) {
      z0 += __bfloat162float(((const __nv_bfloat16 *)ph.bias)[col]);
      z1 += __bfloat162float(((const __nv_bfloat16 *)ph.bias)[col + 1]);
    }
    z0 = act_f(z0, ph.act), z1 = act_f(z1, ph.act);
    if ((sh.ctl->bad_rows >> m) & 1u) z0 = z1 = 0.f;   // out-of-range type: the row's output is defined to be zero
    if (ph.out_bf16) {
      __nv_bfloat162 v = __floats2bfloat162_rn(z0, z1);
      *(uint32_t *)((__nv_bfloat16 *)ph.out + (int64_t)m * ph.out_ld + col) = *(uint32_t *)&v;
    } else {
      *(float2 *)((float *)ph.out + (int64_t)m * ph.out_ld + col) = make_float2(z0, z1);
    }
  }
  return true;
}
// NTU / NTD: 8-column tiles of the up / down strip (compile-time, so that every kernel gets the
// registers its own shape needs).
template <int NTU, int NTD>
__global__ void __launch_bounds__(kThreads, 2) ffn_decode_kernel(const FfnDecodeArgs a) {
  // the next launch of the stream may start now: it only requests its own weights before it waits
  // (triggering later -- after the up phase or after the exchange -- was measured no faster)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 127) & ~(uintptr_t)127);
  uint8_t *wd_sm = smem;                        // W_down slice  [F][sd]
  uint8_t *wu_sm = smem + a.off_wu;             // W_up slice    [D][su]; later part of the H stage
  uint8_t *st_sm = smem + a.off_stage;          // X stage; the H stage starts at wu_sm and runs through here
  Ctl *ctl = (Ctl *)(smem + a.off_ctl);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int c = blockIdx.x, q = a.q, M = a.M;
  const bool has_up = c < a.n_up, has_dn = c < a.n_dn;
  const int col_u = c * a.su, col_d = c * a.sd;
  const int D = a.D, F = a.F;
  ALG_TRACE_VARS;
#define TR(tag) do { if (tid == 0) ALG_TRACE(0, tag); ALG_TRACE_SEQ(tag); } while (0)
  TR(1);

  // ---- tables, barriers ----
  if (a.small_q) {
    for (int e = tid; e <= q; e += kThreads) ctl->so_d[e] = a.so_d[e], ctl->so_f[e] = a.so_f[e];
  } else {
    for (int e = tid; e <= q; e += kThreads) ctl->so_d[e] = a.tab_up->so[e], ctl->so_f[e] = a.tab_dn->so[e];
  }
  const uint32_t bar_up = smem_u32(&ctl->bar_up), bar_dn = smem_u32(&ctl->bar_dn);
  const uint32_t bar_miss = smem_u32(&ctl->bar_miss), bar_x = smem_u32(&ctl->bar_x);
  if (tid == 0) {
    mbar_init(bar_up, kLoaders);        // every loader thread arrives once its copies have landed
    mbar_init(bar_dn, kLoaders);
    mbar_init(bar_miss, 2 * kLoaders);
    mbar_init(bar_x, kStagers);
    ctl->abort_flag = 0;
    ctl->go = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  int spec_type = -1;
  if (tid < M) {   // speculative: the previous kernel may still be writing the types
    spec_type = a.types ? __ldcg(a.types + tid) : (tid % q);
    if (spec_type < 0 || spec_type >= q) spec_type = -1;
  }
  __syncthreads();
  // output groups of the two strips (a strip never straddles groups: su | every f width, sd | every d width)
  int ju = -1, jd = -1;
  if (has_up) {
    ju = 0;
    while (ju + 1 < q && ctl->so_f[ju + 1] <= col_u) ++ju;   // hidden columns are the outputs of up = the inputs of down
  }
  if (has_dn) {
    jd = 0;
    while (jd + 1 < q && ctl->so_d[jd + 1] <= col_d) ++jd;
  }
  if (warp == 0) derive_masks(ctl, a, spec_type, M, q, ju, jd, lane);
  __syncthreads();
  const uint32_t spec_up = ctl->need_up, spec_dn = ctl->need_dn;

  // Requests the rows of the input groups in `mask` of one weight slice: `cols` columns starting at
  // col0, 16 bytes per copy, neighbouring lanes on neighbouring pieces of a row.  t = index of the
  // thread among the `kLoaders` threads of this slice.
  auto request_slice = [&](const __nv_bfloat16 *W, int ld, uint32_t dst, const int *so, uint32_t mask, int col0, int cols,
                           int t) {
    const int ppr = cols >> 3;   // 16-byte pieces per row
    // piece e of a group = (row e / ppr, piece e % ppr); a thread steps by kLoaders pieces at a time,
    // i.e. by (kLoaders / ppr) rows and (kLoaders % ppr) pieces: no division inside the loops
    const int dr = kLoaders / ppr, dp = kLoaders % ppr;
    const int tr0 = t / ppr, tp0 = t % ppr;
    for (int k = 0; k < q; ++k) {
      if (!((mask >> k) & 1u)) continue;
      const int r0 = so[k], rows = so[k + 1] - r0;
      int r = tr0, pc = tp0;
      while (r < rows) {
        cp_async_16_l2line(dst + (uint32_t)(((r0 + r) * ppr + pc) << 4), W + (int64_t)(r0 + r) * ld + col0 + pc * 8);
        r += dr, pc += dp;
        if (pc >= ppr) pc -= ppr, ++r;
      }
    }
  };
  // ---- both weight slices, requested before anything else is waited for ----
  if (tid < kLoaders) {
    if (has_up) request_slice((const __nv_bfloat16 *)a.W_up, F, smem_u32(wu_sm), ctl->so_d, spec_up, col_u, a.su, tid);
    if (!(a.extra_expect_bytes && tid == 0)) cp_async_arrive(bar_up);   // test aid: one arrival short, the barrier never completes
  } else if (tid < 2 * kLoaders) {
    if (has_dn) request_slice((const __nv_bfloat16 *)a.W_down, D, smem_u32(wd_sm), ctl->so_f, spec_dn, col_d, a.sd, tid - kLoaders);
    cp_async_arrive(bar_dn);
  }
  TR(2);
  // ---- everything below may depend on the previous kernel of the stream ----
  asm volatile("griddepcontrol.wait;" ::: "memory");
  TR(3);

  Shared sh;
  sh.ctl = ctl, sh.p_sm = (float *)(smem + a.off_p), sh.bar_x = bar_x;
  sh.M = M, sh.m_pad = a.m_pad, sh.q = q, sh.wait_limit = a.wait_limit, sh.status = a.status;
  Phase up;
  up.src = (const __nv_bfloat16 *)a.X, up.ld = D, up.K = D, up.kc = a.kc_up, up.pitch_bytes = a.kc_up * 2;
  up.stage_base = smem_u32(st_sm), up.w_base = smem_u32(wu_sm), up.cols = a.su, up.col0 = col_u;
  up.so = ctl->so_d, up.rows_k = ctl->rows_up, up.bias = a.b_up, up.act = a.act;
  up.out = a.H, up.out_ld = F, up.out_bf16 = 1, up.first_chunk_staged = true;
  uint32_t x_parity = 0;
  if (has_up) stage_chunk(sh, up, 0, min(a.kc_up, D));
  // the row types as the previous kernel left them: the ones that count
  int my_type = -1;
  if (tid < M) {
    my_type = a.types ? __ldcg(a.types + tid) : (tid % q);
    if (my_type < 0 || my_type >= q) {
      atomicExch(a.status, (int)ALG_ERR_BAD_TYPE);
      my_type = -1;
    }
  }
  if (warp == 0) {
    if (__any_sync(0xffffffffu, my_type != spec_type)) derive_masks(ctl, a, my_type, M, q, ju, jd, lane);
    __syncwarp();
    if (lane == 0) ctl->miss_up = ctl->need_up & ~spec_up, ctl->miss_dn = ctl->need_dn & ~spec_dn;
  }
  __syncthreads();   // final masks visible
  const bool missed = (ctl->miss_up | ctl->miss_dn) != 0u;
  if (missed) {   // rare: blocks the final types need and the early request did not cover
    if (tid < kLoaders) {
      if (has_up) request_slice((const __nv_bfloat16 *)a.W_up, F, smem_u32(wu_sm), ctl->so_d, ctl->miss_up, col_u, a.su, tid);
      cp_async_arrive(bar_miss);
    } else if (tid < 2 * kLoaders) {
      if (has_dn) request_slice((const __nv_bfloat16 *)a.W_down, D, smem_u32(wd_sm), ctl->so_f, ctl->miss_dn, col_d, a.sd, tid - kLoaders);
      cp_async_arrive(bar_miss);
    }
  }
  TR(4);
  bool ok = true;

  // ---------------- up phase: H[:, strip] = act(X *_q W_up + b_up) ----------------
  if (has_up) {
    ok = wait_bar(sh, bar_up, 0);
    if (ok && missed) ok = wait_bar(sh, bar_miss, 0);
    TR(5);
    up.need = ctl->need_up;
    if (ok) ok = run_phase_t<NTU>(sh, up, x_parity);
    TR(6);
    // publish: every thread's H stores become visible device-wide, then one arrival per CTA
    __threadfence();
    __syncthreads();
    if (tid == 0 && ok) atomicAdd(a.counters, 1u);
  }
  if (has_dn) {
    // ---------------- exchange: all of H must be there ----------------
    if (tid == 0) {
      const long long t0 = clock64();
      int go = ctl->abort_flag ? 0 : 1;
      while (go && ld_acquire_u32(a.counters) < (unsigned)a.n_up) {
        if (clock64() - t0 > a.wait_limit) {
          atomicExch(a.status, (int)ALG_ERR_DEVICE_TIMEOUT);
          ctl->abort_flag = 1;
          go = 0;
        }
      }
      ctl->go = go;
    }
    __syncthreads();   // also: every warp is done with the W_up slice and the partial-sum buffer
    ok = ctl->go != 0;
    // the last consumer past the wait clears the counters: the next launch starts from zero
    if (tid == 0 && ok && atomicAdd(a.counters + 1, 1u) == (unsigned)(a.n_dn - 1)) a.counters[0] = 0u, a.counters[1] = 0u;
    TR(7);
    // ---------------- down phase: Y[:, strip] = H *_q W_down + b_down ----------------
    if (ok) {
      Phase dn;
      dn.src = (const __nv_bfloat16 *)a.H, dn.ld = F, dn.K = F, dn.kc = a.kc_dn, dn.pitch_bytes = a.kc_dn * 2;
      dn.stage_base = smem_u32(wu_sm), dn.w_base = smem_u32(wd_sm), dn.cols = a.sd, dn.col0 = col_d;
      dn.so = ctl->so_f, dn.rows_k = ctl->rows_dn, dn.need = ctl->need_dn, dn.bias = a.b_down, dn.act = ALG_ACT_NONE;
      dn.out = a.Y, dn.out_ld = D, dn.out_bf16 = a.y_bf16, dn.first_chunk_staged = true;
      stage_chunk(sh, dn, 0, min(a.kc_dn, F));   // H travels while the weight barrier is checked
      ok = wait_bar(sh, bar_dn, 0);
      if (ok && missed && !has_up) ok = wait_bar(sh, bar_miss, 0);
      TR(8);
      if (ok) ok = run_phase_t<NTD>(sh, dn, x_parity);
    }
  }
  TR(9);
  if (ctl->abort_flag) {  // copies that are still in flight get time to land before shared memory is released
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000LL) {
    }
  }
#undef TR
}

int gcd_i(int x, int y) {
  while (y) {
    const int t = x % y;
    x = y, y = t;
  }
  return x;
}

// smallest strip width (multiple of 8 that divides every group width) that needs at most num_sms CTAs
int pick_strip(int q, const int *w, int total, int num_sms) {
  int g = 0;
  for (int k = 0; k < q; ++k) g = gcd_i(g, w[k]);
  for (int s = 8; s <= 64; s += 8)
    if (g % s == 0 && total / s <= num_sms) return s;
  return 0;
}
// the instantiated strip widths: up to 32 hidden columns and 16 output columns per CTA
void (*pick_kernel(int ntu, int ntd))(const FfnDecodeArgs) {
  if (ntd == 1) {
    if (ntu == 1) return ffn_decode_kernel<1, 1>;
    if (ntu == 2) return ffn_decode_kernel<2, 1>;
    if (ntu == 3) return ffn_decode_kernel<3, 1>;
    if (ntu == 4) return ffn_decode_kernel<4, 1>;
  } else if (ntd == 2) {
    if (ntu == 1) return ffn_decode_kernel<1, 2>;
    if (ntu == 2) return ffn_decode_kernel<2, 2>;
    if (ntu == 3) return ffn_decode_kernel<3, 2>;
    if (ntu == 4) return ffn_decode_kernel<4, 2>;
  }
  return nullptr;
}

}  // namespace

bool ffn_decode_plan(int q, const int *dw, const int *fw, int D, int F, int num_sms, FfnDecodePlan *plan) {
  for (int k = 0; k < q; ++k)
    if (dw[k] % 16 || fw[k] % 16) return false;
  FfnDecodePlan p = {};
  p.su = pick_strip(q, fw, F, num_sms);
  p.sd = pick_strip(q, dw, D, num_sms);
  if (!p.su || !p.sd || !pick_kernel(p.su >> 3, p.sd >> 3)) return false;
  p.n_up = F / p.su, p.n_dn = D / p.sd;
  p.wd_bytes = F * p.sd * 2;
  p.wu_bytes = D * p.su * 2;
  p.p_bytes = kWarps * 16 * (p.su > p.sd ? p.su : p.sd) * 4;   // for 16 staged rows; half of it for 8
  p.ctl_bytes = ((int)sizeof(Ctl) + 127) & ~127;
  p.stage_bytes = kSmemBudget - 128 - p.wd_bytes - p.wu_bytes - p.p_bytes - p.ctl_bytes;
  p.stage_bytes &= ~127;
  if (p.stage_bytes < 16 * 64 * 2) return false;   // at least one 64-deep chunk of 16 rows
  *plan = p;
  return true;
}

cudaError_t launch_ffn_decode(const FfnDecodeArgs &args, const FfnDecodePlan &p, cudaStream_t st) {
  void (*kernel)(const FfnDecodeArgs) = pick_kernel(p.su >> 3, p.sd >> 3);
  if (!kernel) return cudaErrorInvalidConfiguration;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
  if (e != cudaSuccess) return e;
  FfnDecodeArgs a = args;
  a.su = p.su, a.sd = p.sd, a.n_up = p.n_up, a.n_dn = p.n_dn;
  a.m_pad = a.M <= 8 ? 8 : 16;
  // the partial-sum buffer shrinks with the staged rows; what it gives up goes to the activation stage
  const int p_bytes = p.p_bytes * a.m_pad / 16;
  const int stage_bytes = p.stage_bytes + (p.p_bytes - p_bytes);
  a.off_wu = p.wd_bytes;
  a.off_stage = a.off_wu + p.wu_bytes;
  a.off_p = a.off_stage + stage_bytes;
  a.off_ctl = a.off_p + p_bytes;
  auto round64 = [](int v) { return (v + 63) & ~63; };
  a.kc_up = std::min(round64(a.D), (stage_bytes / (a.m_pad * 2)) & ~63);
  a.kc_dn = std::min(round64(a.F), ((p.wu_bytes + stage_bytes) / (a.m_pad * 2)) & ~63);
  if (a.kc_up < 64 || a.kc_dn < 64) return cudaErrorInvalidConfiguration;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(std::max(a.n_up, a.n_dn), 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = a.off_ctl + p.ctl_bytes + 128;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  e = cudaLaunchKernelEx(&cfg, kernel, a);
  count_launch(1);
  return e;
}

}  // namespace algproj
