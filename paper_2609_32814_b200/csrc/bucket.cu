// Row-type bucketing (Algorithm 1, line "I_i <- {b : tau(p_b) = i}") as a stable permutation.
// No host synchronisation anywhere: the row counts per type never leave the device (the GEMM
// kernels turn the bucket offsets into their tile enumeration themselves).
//
//   M <= 65536: one kernel; every CTA counts the rows before its chunk and overall by itself.
//   larger M:
//   kernel 1 (count):   per-chunk histograms (at most 256 chunks).
//   kernel 2 (scatter): each CTA scans the histograms for the bucket offsets and its own bases,
//                       then perm[offset[t] + base[t] + rank_in_chunk] = row  (stable); CTA 0
//                       publishes the bucket offsets.
//   kernel 3 (gather):  Xb[d,:] = X[perm[d],:]  -- every type becomes a contiguous M-slab.
#include "common.cuh"

namespace algproj {

namespace {

__device__ __forceinline__ int row_type(const BucketArgs &a, int row) {
  int t = a.types ? a.types[row] : (row % a.q);
  return (t < 0 || t >= a.q) ? a.q : t;  // pseudo-type q collects out-of-range rows
}

// Kernel 1: per-chunk histograms of the row types (pseudo-type q = out of range).
__global__ void __launch_bounds__(256) bucket_count_kernel(const BucketArgs a) {
  __shared__ int s_cnt[kMaxQ + 1];
  const int tid = threadIdx.x;
  const int nt = a.q + 1;
  if (tid < nt) s_cnt[tid] = 0;
  __syncthreads();
  const int row_begin = blockIdx.x * a.chunk_rows;
  const int row_end = min(a.M, row_begin + a.chunk_rows);
  for (int row = row_begin + tid; row < row_end; row += 256) {
    int t = row_type(a, row);
    if (t == a.q) atomicExch(a.status, (int)ALG_ERR_BAD_TYPE);
    atomicAdd(&s_cnt[t], 1);
  }
  __syncthreads();
  if (tid < nt) a.chunk_counts[blockIdx.x * nt + tid] = s_cnt[tid];
}

// Kernel 2: every CTA scans the (at most 256) chunk histograms to find the bucket offsets and
// its own base inside each bucket, then places its rows (stable inside a type).  CTA 0 also
// publishes the offsets.
__global__ void __launch_bounds__(256) bucket_scatter_kernel(const BucketArgs a) {
  __shared__ int s_wcnt[8][kMaxQ + 1];
  __shared__ int s_total[kMaxQ + 1];
  __shared__ int s_base[kMaxQ + 1];     // rows of this type in earlier chunks (+ earlier sub-blocks)
  __shared__ int s_offset[kMaxQ + 2];
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
    for (int e = tid; e < 8 * (kMaxQ + 1); e += 256) (&s_wcnt[0][0])[e] = 0;
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
    if (tid < nt) {
      int add = 0;
      for (int w = 0; w < 8; ++w) add += s_wcnt[w][tid];
      s_base[tid] += add;
    }
    __syncthreads();
  }

  if (blockIdx.x == 0)
    for (int t = tid; t <= nt; t += 256) a.hdr->offsets[t] = s_offset[t];
}

// One-kernel variant for M <= 65536: every CTA (1024 threads, 1024 rows) reads all row types itself
// (at most 256 KB from L2) and counts, per type, the rows before its own chunk and the rows overall;
// no histogram array, no second launch.  A warp takes 512 rows at a time with sixteen independent
// loads per lane in flight; the counts live in registers: lane t of every warp owns type t
// (pseudo-type q = out of range), fed by one warp ballot per type and 32 rows.
constexpr int kFusedThreads = 1024;
__global__ void __launch_bounds__(kFusedThreads) bucket_fused_kernel(const BucketArgs a) {
  __shared__ int s_before[32][kMaxQ + 1], s_all[32][kMaxQ + 1];
  __shared__ int s_wcnt[32][kMaxQ + 1];
  __shared__ int s_base[kMaxQ + 1], s_offset[kMaxQ + 2];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nt = a.q + 1;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");  // the row types may come from the previous kernel
  const int row_begin = blockIdx.x * kFusedThreads;
  int before = 0, all = 0;
  const int n_super = (a.M + 511) >> 9;
  if (nt <= 8) {
    // q + 1 <= 8 kinds: every lane keeps its own histogram packed in two 64-bit words (16 bits per
    // kind; a lane sees at most 16 rows per pass and a warp total stays below 2^16), so a pass
    // costs two instructions per row and one shuffle reduction instead of (q+1) ballots per row
    unsigned long long all_lo = 0, all_hi = 0, bef_lo = 0, bef_hi = 0;
    for (int sb = warp; sb < n_super; sb += 32) {
      int tt[16];
#pragma unroll
      for (int u = 0; u < 16; ++u) {
        const int row = sb * 512 + u * 32 + lane;
        tt[u] = row < a.M ? row_type(a, row) : -1;
      }
      unsigned long long lo = 0, hi = 0;
#pragma unroll
      for (int u = 0; u < 16; ++u) {
        const unsigned long long one = tt[u] < 0 ? 0ull : 1ull << ((tt[u] & 3) * 16);
        if (tt[u] < 4) lo += one; else hi += one;
      }
      all_lo += lo, all_hi += hi;
      if (sb * 512 < row_begin) bef_lo += lo, bef_hi += hi;
      if (((sb / 32) & 63) == 63) {  // fold into the 32-bit counters before a 16-bit field can overflow
        for (int d = 16; d > 0; d >>= 1) {
          all_lo += __shfl_xor_sync(0xffffffffu, all_lo, d), all_hi += __shfl_xor_sync(0xffffffffu, all_hi, d);
          bef_lo += __shfl_xor_sync(0xffffffffu, bef_lo, d), bef_hi += __shfl_xor_sync(0xffffffffu, bef_hi, d);
        }
        if (lane < nt) {
          all += (int)(((lane < 4 ? all_lo : all_hi) >> ((lane & 3) * 16)) & 0xFFFF);
          before += (int)(((lane < 4 ? bef_lo : bef_hi) >> ((lane & 3) * 16)) & 0xFFFF);
        }
        all_lo = all_hi = bef_lo = bef_hi = 0;
      }
    }
    for (int d = 16; d > 0; d >>= 1) {
      all_lo += __shfl_xor_sync(0xffffffffu, all_lo, d), all_hi += __shfl_xor_sync(0xffffffffu, all_hi, d);
      bef_lo += __shfl_xor_sync(0xffffffffu, bef_lo, d), bef_hi += __shfl_xor_sync(0xffffffffu, bef_hi, d);
    }
    if (lane < nt) {
      all += (int)(((lane < 4 ? all_lo : all_hi) >> ((lane & 3) * 16)) & 0xFFFF);
      before += (int)(((lane < 4 ? bef_lo : bef_hi) >> ((lane & 3) * 16)) & 0xFFFF);
    }
  } else {
    for (int sb = warp; sb < n_super; sb += 32) {
      int tt[16];
#pragma unroll
      for (int u = 0; u < 16; ++u) {
        const int row = sb * 512 + u * 32 + lane;
        tt[u] = row < a.M ? row_type(a, row) : -1;
      }
      int mine = 0;
#pragma unroll
      for (int u = 0; u < 16; ++u)
        for (int k = 0; k < nt; ++k) {
          const unsigned b = __ballot_sync(0xffffffffu, tt[u] == k);
          if (lane == k) mine += __popc(b);
        }
      all += mine;
      if (sb * 512 < row_begin) before += mine;
    }
  }
  if (lane < nt) s_before[warp][lane] = before, s_all[warp][lane] = all;
  for (int e = tid; e < 32 * (kMaxQ + 1); e += kFusedThreads) (&s_wcnt[0][0])[e] = 0;
  __syncthreads();
  if (tid < nt) {
    int bsum = 0, asum = 0;
    for (int w = 0; w < 32; ++w) bsum += s_before[w][tid], asum += s_all[w][tid];
    s_base[tid] = bsum;
    s_all[0][tid] = asum;
  }
  __syncthreads();
  if (tid == 0) {
    int run = 0;
    for (int t = 0; t < nt; ++t) {
      s_offset[t] = run;
      run += s_all[0][t];
    }
    s_offset[nt] = run;  // == M
  }
  const int row = row_begin + tid;
  const bool live = row < a.M;
  const int t = live ? row_type(a, row) : -1 - lane;  // dead lanes never match each other
  if (live && t == a.q) atomicExch(a.status, (int)ALG_ERR_BAD_TYPE);
  const unsigned peers = __match_any_sync(0xffffffffu, t);
  const int rank_in_warp = __popc(peers & ((1u << lane) - 1u));
  if (live && rank_in_warp == 0) s_wcnt[warp][t] = __popc(peers);
  __syncthreads();
  if (live) {
    int bw = 0;
    for (int w = 0; w < warp; ++w) bw += s_wcnt[w][t];
    a.perm[s_offset[t] + s_base[t] + bw + rank_in_warp] = row;
    if (t == a.q && a.Y) {  // out-of-range type: the row's output is defined to be zero
      char *y = (char *)a.Y + (size_t)row * a.ldy * a.y_elem_bytes;
      for (int e = 0; e < a.N * a.y_elem_bytes; ++e) y[e] = 0;
    }
  }
  if (blockIdx.x == 0)
    for (int t2 = tid; t2 <= nt; t2 += kFusedThreads) a.hdr->offsets[t2] = s_offset[t2];
}

__global__ void __launch_bounds__(256) gather_rows_kernel(const uint4 *__restrict__ X, int64_t ldx_v,
                                                          const int *__restrict__ perm, int M, int vecs,
                                                          uint4 *__restrict__ Xb) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");  // perm comes from the bucketing kernel
  // a warp copies one row at a time, four independent 16-byte loads per lane in flight
  const int lane = threadIdx.x & 31;
  const int warp_global = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int n_warps = (gridDim.x * blockDim.x) >> 5;
  for (int d = warp_global; d < M; d += n_warps) {
    const uint4 *src = X + (int64_t)__ldg(perm + d) * ldx_v;
    uint4 *dst = Xb + (int64_t)d * vecs;
    for (int v0 = lane; v0 < vecs; v0 += 128) {
      uint4 r[4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (v0 + u * 32 < vecs) r[u] = __ldg(src + v0 + u * 32);
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (v0 + u * 32 < vecs) dst[v0 + u * 32] = r[u];
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
}  // namespace

cudaError_t launch_bucket(const BucketArgs &a, cudaStream_t st) {
  if (a.M <= 65536) {  // one kernel: every CTA counts for itself
    count_launch(1);
    return launch_pdl(bucket_fused_kernel, ceil_div(a.M, kFusedThreads), kFusedThreads, st, a);
  }
  const int n_chunks = ceil_div(a.M, a.chunk_rows);
  bucket_count_kernel<<<n_chunks, 256, 0, st>>>(a);
  bucket_scatter_kernel<<<n_chunks, 256, 0, st>>>(a);
  count_launch(2);
  return cudaGetLastError();
}

cudaError_t launch_gather_rows(const void *X, int64_t ldx, const int *perm, int M, int K, int elem_bytes,
                               void *Xb, cudaStream_t st) {
  const int vecs = K * elem_bytes / 16;
  int grid = ceil_div(M, 8);  // eight warps (rows) per CTA
  if (grid > 148 * 8) grid = 148 * 8;
  count_launch(1);
  return launch_pdl(gather_rows_kernel, grid, 256, st, (const uint4 *)X, (int64_t)(ldx * elem_bytes / 16), perm, M, vecs,
                    (uint4 *)Xb);
}

}  // namespace algproj
