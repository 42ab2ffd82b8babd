// SIMT grouped projection: true fp32 FMAs, any group widths.  One CTA computes a 64x64 output
// tile of one (row type i, output group j) pair and sums every kept product x_k W_kj
// (k in B(i,j), Eq. recursive-row-action) in registers before the single store.
// Serves the fp32 problems and bf16 shapes the tensor-core path does not cover.
#include "tile_map.cuh"

namespace algproj {

namespace {

constexpr int TM = 64, TN = 64, TK = 16;

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }

__device__ __forceinline__ float apply_act(float z, int act) {
  if (act == ALG_ACT_GELU_ERF) return 0.5f * z * (1.0f + erff(z * 0.70710678118654752f));
  if (act == ALG_ACT_GELU_TANH) {
    float u = 0.7978845608028654f * (z + 0.044715f * z * z * z);
    return 0.5f * z * (1.0f + tanhf(u));
  }
  return z;
}

template <typename T>
__global__ void __launch_bounds__(256) proj_simt_kernel(const ProjArgs a) {
  __shared__ float As[TK][TM + 1];
  __shared__ float Bs[TK][TN];
  __shared__ int s_rows[TM];
  extern __shared__ __align__(16) unsigned char s_map[];  // tile_map_bytes(n_classes)
  TileMap *tm = reinterpret_cast<TileMap *>(s_map);
  const DevTable *__restrict__ tab = a.tab;
  const int q = a.q;
  tile_map_build(tm, tab, a.st, a.q, a.n_classes, a.offsets, a.cyclic_rows, a.M, a.geom);
  const int n_tiles = tm->total;
  const T *__restrict__ X = (const T *)a.X;
  const T *__restrict__ W = (const T *)a.W;
  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;  // 16 x 16 threads, 4 x 4 outputs each

  for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
    TileRec rec = tile_map_decode(tm, a.geom, tile);
    rec.pair &= 0xFFFF;
    const int j = rec.pair % q;
    const int n_valid = min(TN, tab->ro[j + 1] - rec.n0);
    __syncthreads();
    if (tid < TM) {
      int r = rec.row0 + tid;
      s_rows[tid] = (tid < rec.rows) ? (a.in_perm ? a.in_perm[r] : r) : -1;
    }
    __syncthreads();
    float acc[4][4];
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
      for (int v = 0; v < 4; ++v) acc[u][v] = 0.f;

    const uint32_t mask = tab->keep[rec.pair];
    for (int k = 0; k < q; ++k) {
      if (!((mask >> k) & 1u)) continue;
      const int k_begin = tab->so[k], k_end = tab->so[k + 1];
      for (int k0 = k_begin; k0 < k_end; k0 += TK) {
        // A tile: 64 rows x 16 k  (4 elements per thread), B tile: 16 k x 64 cols
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          int idx = tid + e * 256;
          int r = idx >> 4, kk = idx & 15;
          int src = s_rows[r];
          float v = 0.f;
          if (src >= 0 && k0 + kk < k_end) v = to_f32(X[(int64_t)src * a.ldx + k0 + kk]);
          As[kk][r] = v;
          int kb = idx >> 6, c = idx & 63;
          float w = 0.f;
          if (k0 + kb < k_end && c < n_valid)
            w = to_f32(a.w_kmajor ? W[(int64_t)(rec.n0 + c) * a.ldw + k0 + kb] : W[(int64_t)(k0 + kb) * a.ldw + rec.n0 + c]);
          Bs[kb][c] = w;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < TK; ++kk) {
          float av[4], bv[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) av[u] = As[kk][ty * 4 + u];
#pragma unroll
          for (int v = 0; v < 4; ++v) bv[v] = Bs[kk][tx * 4 + v];
#pragma unroll
          for (int u = 0; u < 4; ++u)
#pragma unroll
            for (int v = 0; v < 4; ++v) acc[u][v] = fmaf(av[u], bv[v], acc[u][v]);
        }
        __syncthreads();
      }
    }
    // epilogue: bias, activation, scatter to the original row order
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      int r = ty * 4 + u;
      if (r >= rec.rows) continue;
      int out_row = a.perm ? a.perm[rec.row0 + r] : rec.row0 + r;
#pragma unroll
      for (int v = 0; v < 4; ++v) {
        int c = tx * 4 + v;
        if (c >= n_valid) continue;
        int col = rec.n0 + c;
        float z = acc[u][v];
        if (a.bias) z += to_f32(((const T *)a.bias)[col]);
        z = apply_act(z, a.act);
        if (a.y_bf16) ((__nv_bfloat16 *)a.Y)[(int64_t)out_row * a.ldy + col] = __float2bfloat16_rn(z);
        else ((float *)a.Y)[(int64_t)out_row * a.ldy + col] = z;
      }
    }
  }
}

}  // namespace

cudaError_t launch_proj_simt(const ProjArgs &a, bool in_bf16, cudaStream_t st) {
  const int grid = 148 * 4;
  const size_t map_bytes = tile_map_bytes(a.n_classes);
  static bool attr = false;
  if (!attr) {
    cudaFuncSetAttribute(proj_simt_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024);
    cudaFuncSetAttribute(proj_simt_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024);
    attr = true;
  }
  if (in_bf16) proj_simt_kernel<__nv_bfloat16><<<grid, 256, map_bytes, st>>>(a);
  else proj_simt_kernel<float><<<grid, 256, map_bytes, st>>>(a);
  count_launch(1);
  return cudaGetLastError();
}

}  // namespace algproj
