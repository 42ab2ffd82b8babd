// Small-M (decode) projection: M <= 64 new rows, weight-bandwidth bound.
//
// Section "One-Token Inference": a decode step applies Algorithm 1 to one new row per sequence,
// typed by its absolute position; the paper notes that this regime needs its own matrix-vector
// style implementation and is limited by weight traffic.  Here every weight block W_kj that some
// row needs (k in B(t_b, j) for a present type t_b) is streamed from HBM exactly once, and blocks
// nobody needs are skipped (a single row of the Q_2 law touches 3 of the 4 blocks).
//
// Decomposition: grid = (N / SN column strips) x (K splits); the `splits` CTAs of a strip form a
// thread-block cluster.  A CTA copies its slice of the bank (its share of the rows of every
// needed input group, SN columns wide) into shared memory with 16-byte asynchronous copies that
// are all in flight at once, stages the matching columns of X (rows that do not use a block are
// staged as zeros, which is how the row-type rule is applied), multiplies with warp-level
// mma.sync (bf16 x bf16 -> fp32) and leaves an M x SN partial sum in shared memory.  The cluster
// then reduces the partial sums through distributed shared memory in a fixed order (deterministic,
// nothing goes through global memory), applies bias / activation and stores Y.
#include <cuda_runtime.h>

#include "common.cuh"

namespace algproj {

namespace {

constexpr int kThreads = 128;
constexpr int kMaxSeg = kMaxQ;

struct Seg {
  int grow0;   // first row of W (= first column of X) of the segment
  int len;     // rows, a multiple of 16
  int loc0;    // first local row inside the CTA's slice
  unsigned long long rows;  // bit b set: row b of X uses this block
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void *src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
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
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ float ld_remote_f32(uint32_t local_addr, uint32_t rank) {
  uint32_t remote;
  float v;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote) : "memory");
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

// Shared-memory images.  W slice: [rows][SN] bf16, 16-byte chunks XOR-swizzled so the 8 rows an
// ldmatrix touches fall into different banks.  X slice: [m_pad][x_pitch] bf16, swizzled likewise.
template <int SN>
__device__ __forceinline__ uint32_t w_off(int row, int chunk) {
  constexpr int kChunks = SN / 8;
  const int sw = (kChunks == 8) ? (row & 7) : ((row >> 1) & 3);
  return (uint32_t)(row * SN * 2 + ((chunk ^ sw) << 4));
}
__device__ __forceinline__ uint32_t x_off(int m, int chunk, int x_pitch_bytes) {
  return (uint32_t)(m * x_pitch_bytes + ((chunk ^ (m & 7)) << 4));
}

template <int SN>
__global__ void __launch_bounds__(kThreads) decode_kernel(const DecodeArgs a) {
  constexpr int NT = SN / 32;          // 8-column n-tiles per warp (4 warps share the strip)
  constexpr int kWChunks = SN / 8;     // 16-byte chunks per W row
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ Seg s_seg[kMaxSeg];
  __shared__ int s_nseg, s_rows, s_type[kDecodeMaxM];
  __shared__ unsigned long long s_bad;

  const DevTable *__restrict__ tab = a.tab;
  const int q = tab->q;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int strip = blockIdx.x, split = blockIdx.y, splits = gridDim.y;
  const int n0 = strip * SN;
  const int M = a.M;
  const int m_tiles = (M + 15) >> 4, m_pad = m_tiles << 4;

  // ---- row types, support of this strip ----
  if (tid < kDecodeMaxM) {
    int t = -1;
    if (tid < M) {
      t = a.types ? a.types[tid] : (tid % q);
      if (t < 0 || t >= q) {
        atomicExch(a.status, (int)ALG_ERR_BAD_TYPE);
        t = -1;
      }
    }
    s_type[tid] = t;
  }
  __syncthreads();
  if (tid == 0) {
    int j = 0;
    while (j + 1 < q && tab->ro[j + 1] <= n0) ++j;
    unsigned long long bad = 0;
    for (int b = 0; b < M; ++b)
      if (s_type[b] < 0) bad |= 1ull << b;
    s_bad = bad;
    int nseg = 0, loc = 0;
    for (int k = 0; k < q; ++k) {
      unsigned long long rows = 0;
      for (int b = 0; b < M; ++b)
        if (s_type[b] >= 0 && ((tab->keep[s_type[b] * q + j] >> k) & 1u)) rows |= 1ull << b;
      if (!rows) continue;  // nobody needs W_kj: it is never read
      const int len = (tab->so[k + 1] - tab->so[k]) / splits;
      s_seg[nseg].grow0 = tab->so[k] + split * len;
      s_seg[nseg].len = len;
      s_seg[nseg].loc0 = loc;
      s_seg[nseg].rows = rows;
      loc += len;
      ++nseg;
    }
    s_nseg = nseg;
    s_rows = loc;
  }
  __syncthreads();
  const int nseg = s_nseg, rows_cta = s_rows;
  const int x_pitch_bytes = ((rows_cta + 63) & ~63) * 2;  // whole groups of eight 16-byte chunks
  uint8_t *w_sm = smem;
  uint8_t *x_sm = w_sm + (size_t)a.w_smem_bytes;
  float *p_sm = (float *)(x_sm + (size_t)a.x_smem_bytes);   // [m_pad][SN] partial sums

  // ---- the weight slice: every 16-byte copy in flight at once ----
  {
    const __nv_bfloat16 *W = (const __nv_bfloat16 *)a.W;
    const uint32_t w_base = smem_u32(w_sm);
    for (int s = 0; s < nseg; ++s) {
      const Seg sg = s_seg[s];
      const int chunks = sg.len * kWChunks;
      for (int c = tid; c < chunks; c += kThreads) {
        const int r = c / kWChunks, ch = c % kWChunks;
        cp_async_16(w_base + w_off<SN>(sg.loc0 + r, ch), W + (int64_t)(sg.grow0 + r) * a.ldw + n0 + ch * 8);
      }
    }
  }
  // ---- the matching columns of X; rows that do not use a block are staged as zeros ----
  {
    const __nv_bfloat16 *X = (const __nv_bfloat16 *)a.X;
    const int xchunks = x_pitch_bytes >> 4;
    for (int s = 0; s < nseg; ++s) {
      const Seg sg = s_seg[s];
      const int seg_chunks = sg.len >> 3;
      for (int e = tid; e < m_pad * seg_chunks; e += kThreads) {
        const int m = e / seg_chunks, ch = e % seg_chunks;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (m < M && ((sg.rows >> m) & 1ull)) v = *(const uint4 *)(X + (int64_t)m * a.ldx + sg.grow0 + ch * 8);
        *(uint4 *)(x_sm + x_off(m, (sg.loc0 >> 3) + ch, x_pitch_bytes)) = v;
      }
    }
    (void)xchunks;
  }
  cp_async_wait_all();
  __syncthreads();

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
  for (int k0 = 0; k0 < rows_cta; k0 += 16) {
    uint32_t b[NT * 2];
    if (NT == 2) {
      uint32_t r4[4];
      const int krow = k0 + (lane & 7) + ((lane >> 3) & 1) * 8;
      ldmatrix_x4_trans(w_base + w_off<SN>(krow, wcol_chunk + (lane >> 4)), r4);
      b[0] = r4[0], b[1] = r4[1], b[NT * 2 - 2] = r4[2], b[NT * 2 - 1] = r4[3];
    } else {
      uint32_t r2[2];
      const int krow = k0 + (lane & 7) + ((lane >> 3) & 1) * 8;
      ldmatrix_x2_trans(w_base + w_off<SN>(krow, wcol_chunk), r2);
      b[0] = r2[0], b[1] = r2[1];
    }
#pragma unroll
    for (int mt = 0; mt < 4; ++mt) {
      if (mt < m_tiles) {
        uint32_t af[4];
        const int m = mt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
        ldmatrix_x4(x_base + x_off(m, (k0 >> 3) + (lane >> 4), x_pitch_bytes), af);
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) mma_bf16(acc[mt][nt], af, b[nt * 2], b[nt * 2 + 1]);
      }
    }
  }
  // ---- partial sums to shared memory ----
  {
    const int g = lane >> 2, t4 = lane & 3;
#pragma unroll
    for (int mt = 0; mt < 4; ++mt) {
      if (mt < m_tiles) {
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          const int col = warp * (SN / 4) + nt * 8 + t4 * 2;
          float *p0 = p_sm + (mt * 16 + g) * SN + col;
          float *p1 = p_sm + (mt * 16 + g + 8) * SN + col;
          p0[0] = acc[mt][nt][0], p0[1] = acc[mt][nt][1];
          p1[0] = acc[mt][nt][2], p1[1] = acc[mt][nt][3];
        }
      }
    }
  }
  __syncthreads();
  if (splits > 1) cluster_sync_all();

  // ---- cluster reduction in split order, bias, activation, store ----
  // element e of the M x SN strip is finished by the CTA with e % splits == split
  {
    const uint32_t p_base = smem_u32(p_sm);
    const unsigned long long bad = s_bad;
    for (int e = split + tid * splits; e < M * SN; e += kThreads * splits) {
      const int m = e / SN, n = e % SN;
      float z = 0.f;
      if (splits > 1) {
        for (int s = 0; s < splits; ++s) z += ld_remote_f32(p_base + (uint32_t)(m * SN + n) * 4u, (uint32_t)s);
      } else {
        z = p_sm[m * SN + n];
      }
      const int col = n0 + n;
      if (a.bias) z += __bfloat162float(((const __nv_bfloat16 *)a.bias)[col]);
      z = act_f(z, a.act);
      if ((bad >> m) & 1ull) z = 0.f;  // out-of-range type: the row's output is defined to be zero
      if (a.y_bf16) ((__nv_bfloat16 *)a.Y)[(int64_t)m * a.ldy + col] = __float2bfloat16_rn(z);
      else ((float *)a.Y)[(int64_t)m * a.ldy + col] = z;
    }
  }
  if (splits > 1) cluster_sync_all();  // partial sums stay readable until every CTA has finished
}

template <int SN>
cudaError_t launch_t(const DecodeArgs &a, size_t smem_bytes, cudaStream_t st) {
  static bool attr = false;
  if (!attr) {
    cudaError_t e = cudaFuncSetAttribute(decode_kernel<SN>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) return e;
    attr = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(a.N / SN, a.splits, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = 1;
  at[0].val.clusterDim.y = a.splits;
  at[0].val.clusterDim.z = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, decode_kernel<SN>, a);
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
      const int rows_max = K / sp;  // worst case: every input group needed by the strip
      const size_t w_bytes = (size_t)rows_max * sn * 2;
      const size_t x_bytes = (size_t)kDecodeMaxM * (((rows_max + 63) & ~63) * 2);
      const size_t p_bytes = (size_t)kDecodeMaxM * sn * 4;
      if (w_bytes + x_bytes + p_bytes > 190 * 1024) continue;
      const int ctas = (N / sn) * sp;
      // prefer filling the machine, then not overshooting it, then the wider strip
      long long score = ctas >= num_sms ? (1000000 - (ctas - num_sms)) * 4 : (long long)ctas * 4;
      score += (sn == 64) ? 1 : 0;
      if (score > best_score) {
        best_score = score;
        best.sn = sn, best.splits = sp;
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
  b.w_smem_bytes = plan.w_smem_bytes;
  b.x_smem_bytes = plan.x_smem_bytes;
  const size_t smem = (size_t)plan.w_smem_bytes + plan.x_smem_bytes + plan.p_smem_bytes;
  cudaError_t e = plan.sn == 64 ? launch_t<64>(b, smem, st) : launch_t<32>(b, smem, st);
  count_launch(1);
  return e;
}

}  // namespace algproj
