// Row-type bucketing: the index sets I_i of Algorithm 1 (all rows of type i), built as one stable
// permutation.  No host synchronisation anywhere: the row counts per type never leave the device
// (the GEMM kernels turn the bucket offsets into their tile enumeration themselves).
//
//   M <= 65536: one kernel of M/1024 CTAs: each histograms its own 1024 rows, publishes the counts,
//               meets the others at a counter (bounded wait) and places its rows.
//   larger M:
//   kernel 1 (count):   per-chunk histograms (at most 256 chunks).
//   kernel 2 (scatter): each CTA scans the histograms for the bucket offsets and its own bases,
//                       then perm[offset[t] + base[t] + rank_in_chunk] = row  (stable); CTA 0
//                       publishes the bucket offsets.
//   kernel 3 (gather):  Xb[d,:] = X[perm[d],:]  -- every type becomes a contiguous M-slab.
#include <algorithm>

#include "common.cuh"
#include "trace.cuh"

namespace algproj {
ALG_TRACE_DEFINE(bucket)

namespace {

__device__ __forceinline__ int row_type(const BucketArgs &a, int row) {
  int t = a.types ? a.types[row] : (row % a.q);
  return (t < 0 || t >= a.q) ? a.q : t;  // pseudo-type q collects out-of-range rows
}

// offsets of the same buckets when each is padded to a multiple of 64 rows
__device__ __forceinline__ void write_pad_offsets(WsHeader *hdr, const int *offset, int q) {
  int run = 0;
  for (int t = 0; t < q; ++t) {
    hdr->pad_offsets[t] = run;
    run += (offset[t + 1] - offset[t] + 63) & ~63;
  }
  hdr->pad_offsets[q] = run;
}

// Kernel 1: per-chunk histograms of the row types (pseudo-type q = out of range).  CAP = largest q + 1
// the instantiation serves: kMaxQ + 1 for table-driven handles, kBigMaxQ + 1 for the large-algebra path.
template <int CAP>
__global__ void __launch_bounds__(256) bucket_count_kernel(const BucketArgs a) {
  __shared__ int s_cnt[CAP];
  const int tid = threadIdx.x;
  const int nt = a.q + 1;
  for (int t = tid; t < nt; t += 256) s_cnt[t] = 0;
  __syncthreads();
  const int row_begin = blockIdx.x * a.chunk_rows;
  const int row_end = min(a.M, row_begin + a.chunk_rows);
  for (int row = row_begin + tid; row < row_end; row += 256) {
    int t = row_type(a, row);
    if (t == a.q) atomicExch(a.status, (int)ALG_ERR_BAD_TYPE);
    atomicAdd(&s_cnt[t], 1);
  }
  __syncthreads();
  for (int t = tid; t < nt; t += 256) a.chunk_counts[blockIdx.x * nt + t] = s_cnt[t];
}

// Kernel 2: every CTA scans the (at most 256) chunk histograms to find the bucket offsets and
// its own base inside each bucket, then places its rows (stable inside a type).  CTA 0 also
// publishes the offsets.
template <int CAP>
__global__ void __launch_bounds__(256) bucket_scatter_kernel(const BucketArgs a) {
  __shared__ int s_wcnt[8][CAP];
  __shared__ int s_total[CAP];
  __shared__ int s_base[CAP];     // rows of this type in earlier chunks (+ earlier sub-blocks)
  __shared__ int s_offset[CAP + 1];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nt = a.q + 1;
  const int n_chunks = gridDim.x;
  for (int t = warp; t < nt; t += 8) {
    int before = 0, total = 0;
    for (int c = lane; c < n_chunks; c += 32) {
      int v = a.chunk_counts[c * nt + t];
      total += v;
      if (c < (int)blockIdx.x) before += v;
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
      before += __shfl_xor_sync(0xffffffffu, before, d);
      total += __shfl_xor_sync(0xffffffffu, total, d);
    }
    if (lane == 0) {
      s_total[t] = total;
      s_base[t] = before;
    }
  }
  __syncthreads();
  if (tid == 0) {
    int run = 0;
    for (int t = 0; t < nt; ++t) {
      s_offset[t] = run;
      run += s_total[t];
    }
    s_offset[nt] = run;  // == M
  }
  __syncthreads();

  const int row_begin = blockIdx.x * a.chunk_rows;
  const int row_end = min(a.M, row_begin + a.chunk_rows);
  for (int r0 = row_begin; r0 < row_end; r0 += 256) {
    for (int e = tid; e < 8 * CAP; e += 256) (&s_wcnt[0][0])[e] = 0;
    __syncthreads();
    const int row = r0 + tid;
    const bool live = row < row_end;
    const int t = live ? row_type(a, row) : -1 - lane;  // dead lanes never match each other
    const unsigned peers = __match_any_sync(0xffffffffu, t);
    const int rank_in_warp = __popc(peers & ((1u << lane) - 1u));
    if (live && rank_in_warp == 0) s_wcnt[warp][t] = __popc(peers);
    __syncthreads();
    if (live) {
      int before = 0;
      for (int w = 0; w < warp; ++w) before += s_wcnt[w][t];
      a.perm[s_offset[t] + s_base[t] + before + rank_in_warp] = row;
      if (t == a.q && a.Y) {  // out-of-range type: the row's output is defined to be zero
        char *y = (char *)a.Y + (size_t)row * a.ldy * a.y_elem_bytes;
        for (int e = 0; e < a.N * a.y_elem_bytes; ++e) y[e] = 0;
      }
    }
    __syncthreads();
    for (int t2 = tid; t2 < nt; t2 += 256) {
      int add = 0;
      for (int w = 0; w < 8; ++w) add += s_wcnt[w][t2];
      s_base[t2] += add;
    }
    __syncthreads();
  }

  if (blockIdx.x == 0) {
    // more than kMaxQ types: the offsets go to the caller's array (the fixed header has no room for them)
    int *offsets = a.big_offsets ? a.big_offsets : a.hdr->offsets;
    for (int t = tid; t <= nt; t += 256) offsets[t] = s_offset[t];
    if (tid == 0 && !a.big_offsets) write_pad_offsets(a.hdr, s_offset, a.q);
  }
}

// One-pass variant for M <= 65536 (at most 64 CTAs of 1024 threads, one row per thread): every row
// type is read exactly once.  A CTA ranks its rows inside their type (warp match + per-warp counts),
// publishes its per-type counts, arrives on a counter and waits (bounded) until every CTA has;
// then it sums the counts of all chunks (bucket offsets) and of the chunks before it (its base)
// and writes perm.  All CTAs are resident together: the grid is far smaller than the machine, and
// the kernel launched after it starts only once every CTA of this one has.  The last CTA past the
// wait clears the counter for the next launch.
//
// CLUSTER (M <= 8192, M <= 16384 where the device takes clusters of 16): the CTAs form one thread-block cluster; the per-type counts stay in shared memory, the
// cluster's hardware barrier replaces the counter and every CTA reads its peers' counts through the cluster's
// shared-memory window -- no round trip to L2 between the ranking and the write of perm.
constexpr int kFusedThreads = 1024;
constexpr int kClusterRows = 8 * kFusedThreads;
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
template <bool CLUSTER>
__global__ void __launch_bounds__(kFusedThreads) bucket_onepass_kernel(const BucketArgs a) {
  __shared__ int s_wcnt[32][kMaxQ + 1];   // rows of type t in warp w; then exclusive prefix over the warps
  __shared__ int s_base[kMaxQ + 1], s_offset[kMaxQ + 2];
  __shared__ int s_tot[kMaxQ + 1];        // CLUSTER: rows of type t in this CTA, read by the peers
  __shared__ int s_go;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nt = a.q + 1;
  const int n_chunks = gridDim.x;
  ALG_TRACE_VARS;
  if (tid == 0) ALG_TRACE(0, 1);
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");  // the row types may come from the previous kernel
  if (tid == 0) ALG_TRACE(0, 2);
  for (int e = tid; e < 32 * (kMaxQ + 1); e += kFusedThreads) (&s_wcnt[0][0])[e] = 0;
  const int row = blockIdx.x * kFusedThreads + tid;
  const bool live = row < a.M;
  const int t = live ? row_type(a, row) : -1 - lane;  // dead lanes never match each other
  if (live && t == a.q) atomicExch(a.status, (int)ALG_ERR_BAD_TYPE);
  const unsigned peers = __match_any_sync(0xffffffffu, t);
  const int rank_in_warp = __popc(peers & ((1u << lane) - 1u));
  if (tid == 0) ALG_TRACE(0, 3);
  __syncthreads();
  if (live && rank_in_warp == 0) s_wcnt[warp][t] = __popc(peers);
  __syncthreads();
  for (int ty = warp; ty < nt; ty += kFusedThreads / 32) {   // exclusive prefix over the warps (lane = warp); the total goes to global memory
    const int v = s_wcnt[lane][ty];
    int incl = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int o = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += o;
    }
    s_wcnt[lane][ty] = incl - v;
    if (lane == 31) {
      if (CLUSTER) {
        s_tot[ty] = incl;
      } else {
        a.chunk_counts[blockIdx.x * nt + ty] = incl;
        __threadfence();
      }
    }
  }
  if (CLUSTER) {
    cluster_sync_all();   // (also orders the shared-memory writes above for this CTA's own threads)
    for (int ty = warp; ty < nt; ty += kFusedThreads / 32) {   // lanes over the CTAs of the cluster (at most 16)
      int v = 0;
      if (lane < n_chunks) {
        uint32_t remote;
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"((uint32_t)__cvta_generic_to_shared(&s_tot[ty])), "r"(lane));
        asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(remote) : "memory");
      }
      int before = lane < (int)blockIdx.x ? v : 0, total = v;
#pragma unroll
      for (int d = 8; d > 0; d >>= 1) {
        before += __shfl_xor_sync(0xffffffffu, before, d);
        total += __shfl_xor_sync(0xffffffffu, total, d);
      }
      if (lane == 0) s_base[ty] = before, s_offset[ty] = total;
    }
    cluster_sync_all();   // no CTA leaves (or overwrites s_tot) while a peer may still read its counts
  } else {
  __syncthreads();
  if (tid == 0) {
    ALG_TRACE(0, 4);
    atomicAdd(a.sync, 1u);
    const long long t0 = clock64();
    int go = 1;
    unsigned v;
    do {
      asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(a.sync) : "memory");
      if (v < (unsigned)n_chunks && clock64() - t0 > a.wait_limit) {
        atomicExch(a.status, (int)ALG_ERR_DEVICE_TIMEOUT);
        go = 0;
        break;
      }
    } while (v < (unsigned)n_chunks);
    s_go = go;
    ALG_TRACE(0, 5);
  }
  __syncthreads();
  if (!s_go) return;
  if (tid == 0 && atomicAdd(a.sync + 1, 1u) == (unsigned)(n_chunks - 1)) a.sync[0] = 0u, a.sync[1] = 0u;
  {   // lanes over the chunks (at most 64); the warps share the types, so that their round trips to L2 overlap
    for (int ty = warp; ty < nt; ty += kFusedThreads / 32) {
      int before = 0, total = 0;
      for (int c = lane; c < n_chunks; c += 32) {
        const int v = __ldcg(a.chunk_counts + c * nt + ty);
        total += v;
        if (c < (int)blockIdx.x) before += v;
      }
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) {
        before += __shfl_xor_sync(0xffffffffu, before, d);
        total += __shfl_xor_sync(0xffffffffu, total, d);
      }
      if (lane == 0) s_base[ty] = before, s_offset[ty] = total;
    }
  }
  __syncthreads();
  }
  if (tid == 0) ALG_TRACE(0, 6);
  if (warp == 0) {   // bucket offsets: exclusive prefix of the totals over the types (nt <= 33: lane 0 takes two)
    const int v0 = lane < nt ? s_offset[lane] : 0, v1 = lane == 0 && nt > 32 ? s_offset[32] : 0;
    int incl = v0;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int o = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += o;
    }
    const int total32 = __shfl_sync(0xffffffffu, incl, 31);
    if (lane < nt) s_offset[lane] = incl - v0;
    if (lane == 0) {
      if (nt > 32) s_offset[32] = total32, s_offset[33] = total32 + v1;
      else s_offset[nt] = total32;   // == M
    }
  }
  __syncthreads();
  if (live) {
    a.perm[s_offset[t] + s_base[t] + s_wcnt[warp][t] + rank_in_warp] = row;
    if (t == a.q && a.Y) {  // out-of-range type: the row's output is defined to be zero
      char *y = (char *)a.Y + (size_t)row * a.ldy * a.y_elem_bytes;
      for (int e = 0; e < a.N * a.y_elem_bytes; ++e) y[e] = 0;
    }
  }
  if (tid == 0) ALG_TRACE(0, 7);
  if (blockIdx.x == 0) {
    for (int t2 = tid; t2 <= nt; t2 += kFusedThreads) a.hdr->offsets[t2] = s_offset[t2];
    if (warp == 1) {   // offsets of the buckets padded to multiples of 64 rows (q <= 32: one lane per type)
      const int v = lane < a.q ? (s_offset[lane + 1] - s_offset[lane] + 63) & ~63 : 0;
      int incl = v;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int o = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += o;
      }
      if (lane < a.q) a.hdr->pad_offsets[lane] = incl - v;
      if (lane == 31) a.hdr->pad_offsets[a.q] = incl;
    }
  }
  if (tid == 0) ALG_TRACE(0, 8);
}

// U = 16-byte loads a lane keeps in flight: 4 for rows of up to 2 KB (more registers would cost occupancy there), 16
// for wider rows (the copy of a wide row is bound by its round trips, one per batch of loads)
template <int U>
__global__ void __launch_bounds__(256) gather_rows_kernel(const uint4 *__restrict__ X, int64_t ldx_v,
                                                          const int *__restrict__ perm, int M, int vecs,
                                                          uint4 *__restrict__ Xb) {
  ALG_TRACE_VARS;
  if (threadIdx.x == 0) ALG_TRACE(1, 1);
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");  // perm comes from the bucketing kernel
  if (threadIdx.x == 0) ALG_TRACE(1, 2);
  // a warp copies one row at a time, U independent 16-byte loads per lane in flight
  const int lane = threadIdx.x & 31;
  const int warp_global = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int n_warps = (gridDim.x * blockDim.x) >> 5;
  for (int d = warp_global; d < M; d += n_warps) {
    const uint4 *src = X + (int64_t)__ldg(perm + d) * ldx_v;
    uint4 *dst = Xb + (int64_t)d * vecs;
    for (int v0 = lane; v0 < vecs; v0 += 32 * U) {
      uint4 r[U];
#pragma unroll
      for (int u = 0; u < U; ++u)
        if (v0 + u * 32 < vecs) r[u] = __ldg(src + v0 + u * 32);
#pragma unroll
      for (int u = 0; u < U; ++u)
        if (v0 + u * 32 < vecs) dst[v0 + u * 32] = r[u];
    }
  }
  if (threadIdx.x == 0) ALG_TRACE(1, 3);
}

// padded row p -> original row (or -1 for a pad row / beyond the last bucket)
__device__ __forceinline__ int padded_source_row(const WsHeader *hdr, const int *perm, int q, int p) {
  int t = 0;
  while (t + 1 < q && hdr->pad_offsets[t + 1] <= p) ++t;
  const int rank = p - hdr->pad_offsets[t];
  const int rows = hdr->offsets[t + 1] - hdr->offsets[t];
  return (p < hdr->pad_offsets[q] && rank < rows) ? perm[hdr->offsets[t] + rank] : -1;
}

__global__ void __launch_bounds__(256) gather_rows_padded_kernel(const uint4 *__restrict__ G, int64_t ldg_v,
                                                                 const WsHeader *__restrict__ hdr,
                                                                 const int *__restrict__ perm, int q, int m_pad, int vecs,
                                                                 uint4 *__restrict__ Gp) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");  // perm and the offsets come from the bucketing kernel
  const int lane = threadIdx.x & 31;
  const int warp_global = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int n_warps = (gridDim.x * blockDim.x) >> 5;
  for (int p = warp_global; p < m_pad; p += n_warps) {
    const int src_row = padded_source_row(hdr, perm, q, p);
    uint4 *dst = Gp + (int64_t)p * vecs;
    for (int v0 = lane; v0 < vecs; v0 += 32) dst[v0] = src_row >= 0 ? __ldg(G + (int64_t)src_row * ldg_v + v0) : make_uint4(0, 0, 0, 0);
  }
}

// XpT[c, p] = X[source(p), c]: 64 padded rows x 64 columns per CTA through shared memory, so that both the
// reads (along c) and the writes (along p) are contiguous.
__global__ void __launch_bounds__(256) gather_transpose_padded_kernel(const __nv_bfloat16 *__restrict__ X, int64_t ldx,
                                                                      const WsHeader *__restrict__ hdr,
                                                                      const int *__restrict__ perm, int q, int m_pad, int K,
                                                                      __nv_bfloat16 *__restrict__ XpT) {
  __shared__ __nv_bfloat16 tile[64][66];
  __shared__ int s_src[64];
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int p0 = blockIdx.x * 64, c0 = blockIdx.y * 64;
  const int tid = threadIdx.x;
  if (tid < 64) s_src[tid] = p0 + tid < m_pad ? padded_source_row(hdr, perm, q, p0 + tid) : -1;
  __syncthreads();
  for (int e = tid; e < 64 * 32; e += 256) {   // 64 rows x 32 column pairs
    const int r = e >> 5, cp = (e & 31) * 2;
    const int src_row = s_src[r];
    __nv_bfloat162 v = __floats2bfloat162_rn(0.f, 0.f);
    if (src_row >= 0 && c0 + cp < K) v = *(const __nv_bfloat162 *)(X + (int64_t)src_row * ldx + c0 + cp);
    tile[r][cp] = v.x, tile[r][cp + 1] = v.y;
  }
  __syncthreads();
  for (int e = tid; e < 64 * 32; e += 256) {   // 64 columns x 32 row pairs
    const int c = e >> 5, rp = (e & 31) * 2;
    if (c0 + c < K && p0 + rp < m_pad) {
      __nv_bfloat162 v;
      v.x = tile[rp][c], v.y = tile[rp + 1][c];
      *(__nv_bfloat162 *)(XpT + (int64_t)(c0 + c) * m_pad + p0 + rp) = v;
    }
  }
}

}  // namespace

namespace {
template <typename... Args>
cudaError_t launch_pdl(void (*kernel)(Args...), int grid, int block, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid, 1, 1);
  cfg.blockDim = dim3(block, 1, 1);
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}
// Column groups of c elements widened to c_pad (zeros), optionally row groups of rs rows widened to rs_pad (zero
// rows); a thread moves 4 elements (8 bytes) of one destination row (blockIdx.y walks the rows).
__global__ void __launch_bounds__(256) pad_groups_kernel(const uint2 *__restrict__ src, int64_t ld_src4, const int *__restrict__ perm,
                                                         int rows_dst, int n_col_groups, int c4, int c_pad4, int rs, int rs_pad,
                                                         uint2 *__restrict__ dst) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");   // perm may come from the previous kernel
  const int w4 = n_col_groups * c_pad4;                 // 8-byte pieces per destination row
  for (int R = blockIdx.y; R < rows_dst; R += gridDim.y) {
    int64_t src_row = R;
    bool row_live = true;
    if (rs > 0) {
      const int gr = R / rs_pad, kr = R - gr * rs_pad;
      row_live = kr < rs;
      src_row = (int64_t)gr * rs + kr;
    } else if (perm) {
      src_row = __ldg(perm + R);
    }
    const uint2 *srow = src + src_row * ld_src4;
    uint2 *drow = dst + (int64_t)R * w4;
    for (int x = blockIdx.x * 256 + threadIdx.x; x < w4; x += gridDim.x * 256) {
      const int gc = x / c_pad4, cc = x - gc * c_pad4;
      drow[x] = (row_live && cc < c4) ? __ldg(srow + gc * c4 + cc) : make_uint2(0u, 0u);
    }
  }
}

}  // namespace

cudaError_t launch_pad_groups(const void *src, int64_t ld_src, const int *perm, int rows_src, int n_col_groups, int c, int c_pad,
                              int rs, int rs_pad, void *dst, cudaStream_t st) {
  if (c % 4 || c_pad % 4 || ld_src % 4 || c_pad < c || (rs > 0 && (rs_pad < rs || rows_src % rs))) return cudaErrorInvalidValue;
  const int rows_dst = rs > 0 ? rows_src / rs * rs_pad : rows_src;
  const int w4 = n_col_groups * (c_pad / 4);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)std::max(1, std::min((w4 + 255) / 256, 8)), (unsigned)std::max(1, std::min(rows_dst, 148 * 8)), 1);
  cfg.blockDim = dim3(256, 1, 1);
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  count_launch(1);
  return cudaLaunchKernelEx(&cfg, pad_groups_kernel, (const uint2 *)src, (int64_t)(ld_src / 4), perm, rows_dst, n_col_groups, c / 4,
                            c_pad / 4, rs, rs_pad, (uint2 *)dst);
}

cudaError_t launch_bucket(const BucketArgs &a, cudaStream_t st) {
  if (a.q > kMaxQ) {   // large-algebra path: two kernels, tables sized for kBigMaxQ types
    if (a.q > kBigMaxQ || !a.big_offsets) return cudaErrorInvalidValue;
    const int n_chunks = ceil_div(a.M, a.chunk_rows);
    bucket_count_kernel<kBigMaxQ + 1><<<n_chunks, 256, 0, st>>>(a);
    bucket_scatter_kernel<kBigMaxQ + 1><<<n_chunks, 256, 0, st>>>(a);
    count_launch(2);
    return cudaGetLastError();
  }
  // clusters of 16 are not portable: asked for once, used where the device says one can be resident
  static int rows16 = -1;
  if (rows16 < 0) {
    rows16 = 0;
    if (cudaFuncSetAttribute(bucket_onepass_kernel<true>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess) {
      cudaLaunchConfig_t probe = {};
      probe.gridDim = dim3(16, 1, 1);
      probe.blockDim = dim3(kFusedThreads, 1, 1);
      cudaLaunchAttribute pa[1];
      pa[0].id = cudaLaunchAttributeClusterDimension;
      pa[0].val.clusterDim.x = 16, pa[0].val.clusterDim.y = 1, pa[0].val.clusterDim.z = 1;
      probe.attrs = pa;
      probe.numAttrs = 1;
      int n = 0;
      if (cudaOccupancyMaxActiveClusters(&n, bucket_onepass_kernel<true>, &probe) == cudaSuccess && n > 0) rows16 = 16 * kFusedThreads;
    }
    (void)cudaGetLastError();
  }
  if (a.M <= std::max(kClusterRows, rows16)) {   // one kernel, one cluster of 1 ... 16 CTAs (CTAs past the batch hold no row)
    int n_cta = 1;
    while (n_cta * kFusedThreads < a.M) n_cta *= 2;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_cta, 1, 1);
    cfg.blockDim = dim3(kFusedThreads, 1, 1);
    cfg.stream = st;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    at[1].id = cudaLaunchAttributeClusterDimension;
    at[1].val.clusterDim.x = n_cta, at[1].val.clusterDim.y = 1, at[1].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 2;
    count_launch(1);
    return cudaLaunchKernelEx(&cfg, bucket_onepass_kernel<true>, a);
  }
  if (a.M <= 65536 && a.sync) {  // one kernel, every row type read once
    count_launch(1);
    return launch_pdl(bucket_onepass_kernel<false>, ceil_div(a.M, kFusedThreads), kFusedThreads, st, a);
  }
  const int n_chunks = ceil_div(a.M, a.chunk_rows);
  bucket_count_kernel<kMaxQ + 1><<<n_chunks, 256, 0, st>>>(a);
  bucket_scatter_kernel<kMaxQ + 1><<<n_chunks, 256, 0, st>>>(a);
  count_launch(2);
  return cudaGetLastError();
}

cudaError_t launch_gather_rows(const void *X, int64_t ldx, const int *perm, int M, int K, int elem_bytes,
                               void *Xb, cudaStream_t st) {
  const int vecs = K * elem_bytes / 16;
  int grid = ceil_div(M, 8);  // eight warps (rows) per CTA
  if (grid > 148 * 8) grid = 148 * 8;
  count_launch(1);
  if (vecs > 128)
    return launch_pdl(gather_rows_kernel<16>, grid, 256, st, (const uint4 *)X, (int64_t)(ldx * elem_bytes / 16), perm, M, vecs,
                      (uint4 *)Xb);
  return launch_pdl(gather_rows_kernel<4>, grid, 256, st, (const uint4 *)X, (int64_t)(ldx * elem_bytes / 16), perm, M, vecs,
                    (uint4 *)Xb);
}

cudaError_t launch_gather_rows_padded(const void *G, int64_t ldg, const WsHeader *hdr, const int *perm, int q, int m_pad,
                                      int N, void *Gp, cudaStream_t st) {
  const int vecs = N * 2 / 16;
  int grid = ceil_div(m_pad, 8);
  if (grid > 148 * 8) grid = 148 * 8;
  count_launch(1);
  return launch_pdl(gather_rows_padded_kernel, grid, 256, st, (const uint4 *)G, (int64_t)(ldg * 2 / 16), hdr, perm, q, m_pad,
                    vecs, (uint4 *)Gp);
}

cudaError_t launch_gather_transpose_padded(const void *X, int64_t ldx, const WsHeader *hdr, const int *perm, int q,
                                           int m_pad, int K, void *XpT, cudaStream_t st) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(ceil_div(m_pad, 64), ceil_div(K, 64), 1);
  cfg.blockDim = dim3(256, 1, 1);
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  count_launch(1);
  return cudaLaunchKernelEx(&cfg, gather_transpose_padded_kernel, (const __nv_bfloat16 *)X, ldx, hdr, perm, q, m_pad, K,
                            (__nv_bfloat16 *)XpT);
}

}  // namespace algproj
