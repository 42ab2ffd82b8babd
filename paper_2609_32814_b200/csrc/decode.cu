// Small-M (decode) projection: M <= 64 new rows, weight-bandwidth bound.
//
// Section "One-Token Inference": a decode step applies Algorithm 1 to one new row per sequence,
// typed by its absolute position; the paper notes that this regime needs its own matrix-vector
// style implementation and is limited by weight traffic.  Here every weight block W_kj that some
// row needs (k in B(t_b, j) for a present type t_b) is streamed from HBM exactly once, and blocks
// nobody needs are skipped (a single row of the Q_2 law touches 3 of the 4 blocks).
//
// Decomposition: grid = (N / SN column strips) x (K splits); the `splits` CTAs of a strip form a
// thread-block cluster.  A CTA fetches its slice of the bank (its share of the rows of every
// needed input group, SN columns wide) with one or two TMA boxes per group -- issued before it
// waits for the previous kernel in the stream (programmatic dependent launch), because weights do
// not depend on it.  Which groups are needed follows from the row types, which MAY come from that
// previous kernel: they are read once before the wait to choose the boxes and once more after it;
// if the second reading differs, the slice is fetched again for the types that count.  It then stages the matching columns of X with 16-byte asynchronous copies (rows
// that do not use a block are staged as zeros, which is how the row-type rule is applied),
// multiplies with warp-level mma.sync (bf16 x bf16 -> fp32), and pushes its partial sums into the
// shared memory of the CTA that owns the output row (row m belongs to CTA m mod splits).  After
// one cluster barrier every CTA adds the partial sums of its rows in split order (deterministic,
// nothing goes through global memory), applies bias / activation and stores Y.
#include <cuda_runtime.h>

#include "tc_common.cuh"

namespace algproj {

using namespace tc;

ALG_TRACE_DEFINE(decode)

namespace {

constexpr int kThreads = 128;
constexpr int kMaxBoxRows = 256;

struct Seg {
  int grow0;   // first row of W (= first column of X) of the segment
  int len;     // rows, a multiple of 16
  int loc0;    // first local row inside the CTA's slice
  uint32_t rows_lo, rows_hi;  // bit b set: row b of X uses this block
};

__device__ __forceinline__ void cp_async_16_zfill(uint32_t dst, const void *src, bool valid) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(valid ? 16 : 0) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() {
  asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x2_trans(uint32_t addr, uint32_t (&r)[2]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0,%1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void st_remote_f32x2(uint32_t local_addr, uint32_t rank, float x, float y) {
  uint32_t remote;
  asm("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
  asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(remote), "f"(x), "f"(y) : "memory");
}
__device__ __forceinline__ float act_f(float z, int act) {
  if (act == ALG_ACT_GELU_ERF) return 0.5f * z * (1.0f + erff(z * 0.70710678118654752f));
  if (act == ALG_ACT_GELU_TANH) {
    float u = 0.7978845608028654f * (z + 0.044715f * z * z * z);
    return 0.5f * z * (1.0f + tanhf(u));
  }
  return z;
}

// Shared-memory images.  W slice: [rows][SN] bf16 as the TMA writes it with its 128-byte (SN = 64)
// or 64-byte (SN = 32) swizzle: 16-byte chunk c of row r sits at chunk c ^ (r & 7), resp.
// c ^ ((r >> 1) & 3), so the 8 rows an ldmatrix touches fall into different banks.  X slice:
// [m_pad][x_pitch] bf16, written by this kernel with the same kind of XOR.
template <int SN>
__device__ __forceinline__ uint32_t w_off(int row, int chunk) {
  constexpr int kChunks = SN / 8;
  const int sw = (kChunks == 8) ? (row & 7) : ((row >> 1) & 3);
  return (uint32_t)(row * SN * 2 + ((chunk ^ sw) << 4));
}
__device__ __forceinline__ uint32_t x_off(int m, int chunk, int x_pitch_bytes) {
  return (uint32_t)(m * x_pitch_bytes + ((chunk ^ (m & 7)) << 4));
}

#define DTR() ALG_TRACE(0, 0)

template <int SN>
__global__ void __launch_bounds__(kThreads) decode_kernel(const __grid_constant__ CUtensorMap tmW, const DecodeArgs a) {
  constexpr int NT = SN / 32;          // 8-column n-tiles per warp (4 warps share the strip)
  extern __shared__ uint8_t smem_raw[];
  __shared__ Seg s_seg[kMaxQ];
  __shared__ int s_nseg, s_rows;
  __shared__ int s_so[kMaxQ + 1], s_ro[kMaxQ + 1];
  __shared__ uint32_t s_keep[kMaxPairs];
  __shared__ uint32_t s_rows32[kMaxQ][2], s_bad32[2];
  __shared__ __align__(8) uint64_t s_bar;

  const DevTable *__restrict__ tab = a.tab;
  const int q = a.q;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int strip = blockIdx.x, split = blockIdx.y, splits = gridDim.y;
  // x / splits = __umulhi(x, a.inv_splits) for every x the kernel divides (below 2^29): no integer division on the way
  const uint32_t inv_splits = a.inv_splits;
  auto div_splits = [&](int x) { return splits == 1 ? x : (int)__umulhi((uint32_t)x, inv_splits); };
  const int n0 = strip * SN;
  const int M = a.M;
  const int m_tiles = (M + 15) >> 4, m_pad = m_tiles << 4;
  ALG_TRACE_VARS;
  DTR();

  // ---- row types, support of this strip (one global round trip, then shared memory only) ----
  if (a.small_q) {  // table travels in the kernel parameters: no global metadata load at all
    for (int e = tid; e <= q; e += kThreads) s_so[e] = a.so[e], s_ro[e] = a.ro[e];
    for (int e = tid; e < q * q; e += kThreads) s_keep[e] = a.keep[e];
  } else {
    for (int e = tid; e <= q; e += kThreads) s_so[e] = tab->so[e], s_ro[e] = tab->ro[e];
    for (int e = tid; e < q * q; e += kThreads) s_keep[e] = tab->keep[e];
  }
  if (tid == 0) {
    mbar_init(smem_u32(&s_bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmW) : "memory");
  }
  int j = 0;
  const uint32_t bar = smem_u32(&s_bar);
  uint8_t *w_sm = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t *x_sm = w_sm + (size_t)a.w_smem_bytes;
  float *r_sm = (float *)(x_sm + (size_t)a.x_smem_bytes);   // [splits][rows owned][SN] partial sums of my rows
  int my_type = -1;
  // Reads the row types (L2, never a stale L1 line), derives the support of this strip and the
  // segment list, and requests the weight slice: one TMA box per segment (more when a segment
  // exceeds the box height).  Runs once before the wait for the previous kernel and, only if the
  // types read after that wait differ, a second time.
  auto plan_and_fetch = [&]() {
    my_type = -1;
    if (tid < M) {
      my_type = a.types ? __ldcg(a.types + tid) : (tid % q);
      if (my_type < 0 || my_type >= q) my_type = -1;
    }
    __syncthreads();   // tables and barrier are ready (first pass); previous segment list is consumed (second pass)
    j = 0;
    while (j + 1 < q && s_ro[j + 1] <= n0) ++j;
    if (tid < kDecodeMaxM) {  // warps 0 and 1: rows 0..63
      const uint32_t kmask = my_type >= 0 ? s_keep[my_type * q + j] : 0u;  // input groups this row uses for group j
      const unsigned badv = __ballot_sync(0xffffffffu, tid < M && my_type < 0);
      if (lane == 0) s_bad32[warp] = badv;
      for (int k = 0; k < q; ++k) {
        const unsigned v = __ballot_sync(0xffffffffu, (kmask >> k) & 1u);
        if (lane == 0) s_rows32[k][warp] = v;
      }
    }
    __syncthreads();
    if (warp == 0) {  // segment list: lane k owns input group k; prefix of the lengths by shuffles
      uint32_t lo = 0, hi = 0;
      int len = 0;
      if (lane < q) {
        lo = s_rows32[lane][0], hi = s_rows32[lane][1];
        if (lo | hi) len = div_splits(s_so[lane + 1] - s_so[lane]);  // nobody needs W_kj -> it is never read
      }
      const unsigned have = __ballot_sync(0xffffffffu, len > 0);
      int incl = len;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += n;
      }
      if (len > 0) {
        const int s = __popc(have & ((1u << lane) - 1u));
        s_seg[s].grow0 = s_so[lane] + split * len;
        s_seg[s].len = len;
        s_seg[s].loc0 = incl - len;
        s_seg[s].rows_lo = lo, s_seg[s].rows_hi = hi;
      }
      if (lane == 31) s_nseg = __popc(have), s_rows = incl;
    }
    __syncthreads();
    if (tid == 0) {
      mbar_expect_tx(bar, (uint32_t)(s_rows * SN * 2 + a.extra_expect_bytes));
      for (int s = 0; s < s_nseg; ++s) {
        const Seg sg = s_seg[s];
        for (int r0 = 0; r0 < sg.len; r0 += a.box_rows)
          tma_load_2d(smem_u32(w_sm) + (uint32_t)((sg.loc0 + r0) * SN * 2), &tmW, bar, n0, sg.grow0 + r0);
      }
    }
  };
  // Bounded wait for the weight slice (parity = phase of the barrier).
  auto wait_weights = [&](uint32_t parity) {
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
      if (clock64() - t0 > a.wait_limit) {
        atomicExch(a.status, (int)ALG_ERR_DEVICE_TIMEOUT);
        while (clock64() - t0 < a.wait_limit + 2000000LL) {  // copies still in flight get time to land
        }
        return false;
      }
    }
    return true;
  };
  plan_and_fetch();
  DTR();
  // The weights do not depend on the previous kernel in the stream, X does: let the next kernel
  // start its own weight stream now, and wait for the producer of X only here.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  DTR();
  uint32_t w_parity = 0;
  bool weights_ok = true;
  {  // the row types as the previous kernel left them: the ones that count
    int t_now = -1;
    if (tid < M) {
      t_now = a.types ? __ldcg(a.types + tid) : (tid % q);
      if (t_now < 0 || t_now >= q) {
        atomicExch(a.status, (int)ALG_ERR_BAD_TYPE);
        t_now = -1;
      }
    }
    if (__syncthreads_or(t_now != my_type)) {
      // fetched for other types than the final ones: let those copies land, then fetch again
      weights_ok = wait_weights(0);
      __syncthreads();
      if (weights_ok) {
        plan_and_fetch();
        w_parity = 1;
      }
    }
  }
  const int nseg = s_nseg, rows_cta = s_rows;
  const int x_pitch_bytes = ((rows_cta + 63) & ~63) * 2;  // whole groups of eight 16-byte chunks
  // ---- the matching columns of X; rows that do not use a block are staged as zeros ----
  {
    const __nv_bfloat16 *X = (const __nv_bfloat16 *)a.X;
    const uint32_t x_base = smem_u32(x_sm);
    // thread -> (row m = tid / 8 + 16 i, chunk ch = tid % 8 + 8 jj): no divisions in the loop
    const int m_lo = tid >> 3, ch_lo = tid & 7;
    for (int s = 0; s < nseg; ++s) {
      const Seg sg = s_seg[s];
      const int seg_chunks = sg.len >> 3;
      for (int m = m_lo; m < m_pad; m += kThreads / 8) {
        const bool use = m < M && (((m < 32 ? sg.rows_lo : sg.rows_hi) >> (m & 31)) & 1u);
        const __nv_bfloat16 *src = X + (int64_t)(use ? m : 0) * a.ldx + sg.grow0;
        for (int ch = ch_lo; ch < seg_chunks; ch += 8)
          cp_async_16_zfill(x_base + x_off(m, (sg.loc0 >> 3) + ch, x_pitch_bytes), src + ch * 8, use);
      }
    }
  }
  DTR();
  cp_async_wait_all();
  if (weights_ok) wait_weights(w_parity);   // on expiry: status raised, the result is invalid, the kernel still ends
  __syncthreads();
  DTR();

  // ---- warp-level MMA: warp w owns columns [w * SN/4, +SN/4) of the strip, all rows ----
  float acc[4][NT][4];
#pragma unroll
  for (int mt = 0; mt < 4; ++mt)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[mt][nt][e] = 0.f;
  const uint32_t w_base = smem_u32(w_sm), x_base = smem_u32(x_sm);
  const int wcol_chunk = warp * (SN / 32);  // first 16-byte chunk of this warp's columns
  const int frag_row = (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll 2
  for (int k0 = 0; k0 < rows_cta; k0 += 16) {
    uint32_t b[4];
    if (NT == 2) {
      ldmatrix_x4_trans(w_base + w_off<SN>(k0 + frag_row, wcol_chunk + (lane >> 4)), b);
    } else {
      uint32_t r2[2];
      ldmatrix_x2_trans(w_base + w_off<SN>(k0 + frag_row, wcol_chunk), r2);
      b[0] = r2[0], b[1] = r2[1], b[2] = 0, b[3] = 0;
    }
    uint32_t af[4][4];
#pragma unroll
    for (int mt = 0; mt < 4; ++mt)
      if (mt < m_tiles) ldmatrix_x4(x_base + x_off(mt * 16 + frag_row, (k0 >> 3) + (lane >> 4), x_pitch_bytes), af[mt]);
#pragma unroll
    for (int mt = 0; mt < 4; ++mt)
      if (mt < m_tiles) {
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) mma_bf16(acc[mt][nt], af[mt], b[nt * 2], b[nt * 2 + 1]);
      }
  }
  DTR();
  // ---- push the partial sums to the owners of the rows: row m -> CTA m % splits, slot m / splits ----
  const int rows_owned_max = div_splits(m_pad + splits - 1);
  {
    const uint32_t r_base = smem_u32(r_sm);
    const int g = lane >> 2, t4 = lane & 3;
#pragma unroll
    for (int mt = 0; mt < 4; ++mt) {
      if (mt < m_tiles) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int m = mt * 16 + g + h * 8;
          const int slot = div_splits(m);
          const uint32_t owner = (uint32_t)(m - slot * splits);
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            const int col = warp * (SN / 4) + nt * 8 + t4 * 2;
            const uint32_t off = r_base + (uint32_t)(((split * rows_owned_max + slot) * SN + col) * 4);
            if (splits > 1) st_remote_f32x2(off, owner, acc[mt][nt][h * 2], acc[mt][nt][h * 2 + 1]);
            else *(float2 *)(r_sm + (slot * SN + col)) = make_float2(acc[mt][nt][h * 2], acc[mt][nt][h * 2 + 1]);
          }
        }
      }
    }
  }
  if (splits > 1) cluster_sync_all();  // all partial sums of my rows have arrived; no remote access after this
  else __syncthreads();
  DTR();

  // ---- add the partial sums of my rows in split order, bias, activation, store ----
  {
    constexpr int kGroups = SN / 4;
    const int my_rows = div_splits(M - split + splits - 1);  // rows m = split + splits * slot < M
    for (int e = tid; e < my_rows * kGroups; e += kThreads) {
      const int slot = e / kGroups, n = (e % kGroups) * 4;
      const int m = split + slot * splits;
      float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int s = 0; s < splits; ++s) {
        const float4 p = *(const float4 *)(r_sm + ((s * rows_owned_max + slot) * SN + n));
        z.x += p.x, z.y += p.y, z.z += p.z, z.w += p.w;
      }
      const int col = n0 + n;
      const bool bad = ((m < 32 ? s_bad32[0] : s_bad32[1]) >> (m & 31)) & 1u;
      float v[4] = {z.x, z.y, z.z, z.w};
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        if (a.bias) v[c] += __bfloat162float(((const __nv_bfloat16 *)a.bias)[col + c]);
        v[c] = act_f(v[c], a.act);
        if (bad) v[c] = 0.f;  // out-of-range type: the row's output is defined to be zero
      }
      if (a.y_bf16) {
        __nv_bfloat162 lo = __floats2bfloat162_rn(v[0], v[1]), hi = __floats2bfloat162_rn(v[2], v[3]);
        *(uint2 *)((__nv_bfloat16 *)a.Y + (int64_t)m * a.ldy + col) = make_uint2(*(uint32_t *)&lo, *(uint32_t *)&hi);
      } else {
        *(float4 *)((float *)a.Y + (int64_t)m * a.ldy + col) = make_float4(v[0], v[1], v[2], v[3]);
      }
    }
  }
  DTR();
}

template <int SN>
cudaError_t launch_t(const DecodeArgs &a, size_t smem_bytes, cudaStream_t st) {
  static bool attr = false;
  if (!attr) {
    cudaError_t e = cudaFuncSetAttribute(decode_kernel<SN>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) return e;
    attr = true;
  }
  CUtensorMap tmW;
  cudaError_t e = make_map_2d_sw(&tmW, a.W, (uint64_t)a.N, (uint64_t)a.K, (uint64_t)a.ldw * 2, SN, (uint32_t)a.box_rows,
                                 SN * 2);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(a.N / SN, a.splits, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = st;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = 1;
  at[0].val.clusterDim.y = a.splits;
  at[0].val.clusterDim.z = 1;
  // programmatic dependent launch: this kernel may start while its predecessor in the stream is
  // still running; it waits (griddepcontrol.wait) before touching anything the predecessor writes
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, decode_kernel<SN>, tmW, a);
}

}  // namespace

// Chooses the strip width and the K split for a projection with input widths s[q], N columns:
// as many CTAs as SMs or a little more, clusters of at most 8, slices that fit shared memory.
bool decode_plan(int q, const int *s, int K, int N, int num_sms, DecodePlan *plan) {
  int g = 0;  // gcd of s[k] / 16
  for (int k = 0; k < q; ++k) {
    if (s[k] % 16) return false;
    int v = s[k] / 16;
    while (v) { int t = g % v; g = v; v = t; }
  }
  if (g == 0) return false;
  DecodePlan best = {};
  long long best_score = -1;
  for (int sn = 64; sn >= 32; sn -= 32) {
    if (N % sn) continue;
    for (int sp = 1; sp <= 8; ++sp) {
      if (g % sp) continue;
      // one TMA box per segment piece: rows per box divide every s[k] / sp, at most 256
      int box = 0;
      for (int k = 0; k < q; ++k) {
        int v = s[k] / sp;
        int t = box;
        while (v) { int u = t % v; t = v; v = u; }
        box = t;
      }
      while (box > kMaxBoxRows) box /= 2;
      if (box % 8) continue;
      const int rows_max = K / sp;  // worst case: every input group needed by the strip
      const size_t w_bytes = (size_t)rows_max * sn * 2;
      const size_t x_bytes = (size_t)kDecodeMaxM * (((rows_max + 63) & ~63) * 2);
      const size_t p_bytes = (size_t)(kDecodeMaxM + 8) * sn * 4;
      if (w_bytes + x_bytes + p_bytes + 1024 > 190 * 1024) continue;
      const int ctas = (N / sn) * sp;
      // prefer filling the machine, then not overshooting it, then the wider strip
      long long score = ctas >= num_sms ? (1000000 - (ctas - num_sms)) * 4 : (long long)ctas * 4;
      score += (sn == 64) ? 1 : 0;
      if (score > best_score) {
        best_score = score;
        best.sn = sn, best.splits = sp, best.box_rows = box;
        best.w_smem_bytes = (int)w_bytes, best.x_smem_bytes = (int)x_bytes, best.p_smem_bytes = (int)p_bytes;
      }
    }
  }
  if (best_score < 0) return false;
  *plan = best;
  return true;
}

cudaError_t launch_decode(const DecodeArgs &a, const DecodePlan &plan, cudaStream_t st) {
  DecodeArgs b = a;
  b.splits = plan.splits;
  b.inv_splits = (uint32_t)((0x100000000ull + (uint64_t)plan.splits - 1) / (uint64_t)plan.splits);
  b.box_rows = plan.box_rows;
  b.w_smem_bytes = plan.w_smem_bytes;
  b.x_smem_bytes = plan.x_smem_bytes;
  const size_t smem = (size_t)plan.w_smem_bytes + plan.x_smem_bytes + plan.p_smem_bytes + 1024;
  cudaError_t e = plan.sn == 64 ? launch_t<64>(b, smem, st) : launch_t<32>(b, smem, st);
  count_launch(1);
  return e;
}

}  // namespace algproj
