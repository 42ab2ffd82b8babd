// PTX wrappers and small device helpers shared by the tensor-core kernels (sm_100a only).
#pragma once

#include <cuda.h>

#include "tile_map.cuh"
#include "trace.cuh"

namespace algproj {
namespace tc {

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
// Four rows of a 2-D tensor (row coordinates r0..r3, box {columns, 1}) land as four consecutive rows of the
// destination, swizzled like a tiled box.
__device__ __forceinline__ void tma_gather4(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int r0, int r1, int r2,
                                            int r3) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, "
      "%7}], [%2];" ::"r"(dst),
      "l"(map), "r"(bar), "r"(c0), "r"(r0), "r"(r1), "r"(r2), "r"(r3)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];" ::"r"(
          dst),
      "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1, int c2,
                                            int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];" ::"r"(
          dst),
      "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
// One lane of the (converged) warp; the choice is uniform-friendly, unlike `lane == 0`.
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "elect.sync _|p, 0xffffffff;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(pred));
  return pred != 0;
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

// Tiled stores shared -> global (bulk async group of the issuing thread).
__device__ __forceinline__ void tma_store_2d(uint32_t src_smem, const CUtensorMap *map, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(map), "r"(src_smem),
               "r"(x), "r"(y)
               : "memory");
}
__device__ __forceinline__ void tma_store_3d(uint32_t src_smem, const CUtensorMap *map, int x, int y, int z) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];" ::"l"(map),
               "r"(src_smem), "r"(x), "r"(y), "r"(z)
               : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Shared-memory matrix descriptor (sm_100 format): start address, leading / stride byte
// offsets (all >> 4), descriptor version 1, swizzle mode (2 = 128-byte, 4 = 64-byte atoms).
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes,
                                                   uint64_t swizzle_mode = 2) {
  uint64_t d = (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= 1ull << 46;
  d |= swizzle_mode << 61;
  return d;
}

// GELU with the exact (erf) definition, gelu(z) = z * Phi(z) = max(z, 0) - |z| * Phi(-|z|).  The
// lower tail Phi(-u), u >= 0, is evaluated as 2^p(u) with a degree-6 polynomial p fitted to
// log2(Phi(-u)) on [0, 6] (one ex2, no branches); |gelu error| < 1e-7 over the whole real line,
// i.e. fp32 rounding level.  Two values are processed at once with the packed fp32x2 FMA of
// sm_100, which halves the issue slots the epilogue takes from the producer and MMA threads.
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  return (uint64_t)__float_as_uint(lo) | ((uint64_t)__float_as_uint(hi) << 32);
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ void gelu_erf2(float &z0, float &z1) {
  const float u0 = fminf(fabsf(z0), 6.0f), u1 = fminf(fabsf(z1), 6.0f);
  const uint64_t u = pack2(u0, u1);
  uint64_t p = pack2(3.3093889e-05f, 3.3093889e-05f);
  p = fma2(p, u, pack2(-7.6922908e-04f, -7.6922908e-04f));
  p = fma2(p, u, pack2(8.0807470e-03f, 8.0807470e-03f));
  p = fma2(p, u, pack2(-5.3412151e-02f, -5.3412151e-02f));
  p = fma2(p, u, pack2(-4.5877093e-01f, -4.5877093e-01f));
  p = fma2(p, u, pack2(-1.1512017f, -1.1512017f));
  p = fma2(p, u, pack2(-0.99999309f, -0.99999309f));
  float t0, t1;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(t0) : "f"(__uint_as_float((uint32_t)p)));
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(t1) : "f"(__uint_as_float((uint32_t)(p >> 32))));
  z0 = fmaf(-fabsf(z0), t0, fmaxf(z0, 0.0f));
  z1 = fmaf(-fabsf(z1), t1, fmaxf(z1, 0.0f));
}
__device__ __forceinline__ float gelu_tanh(float z) {
  float u = 0.7978845608028654f * (z + 0.044715f * z * z * z);
  return 0.5f * z * (1.0f + tanhf(u));
}


// Bias and activation on one row segment of 32 fp32 accumulator values.
__device__ __forceinline__ void finish_32(float (&f)[32], const ProjArgs &a, int col) {
  if (a.bias) {
    const __nv_bfloat16 *b = (const __nv_bfloat16 *)a.bias + col;
#pragma unroll
    for (int x = 0; x < 32; ++x) f[x] += __bfloat162float(__ldg(b + x));
  }
  if (a.act == ALG_ACT_GELU_ERF) {
#pragma unroll
    for (int x = 0; x < 32; x += 2) gelu_erf2(f[x], f[x + 1]);
  } else if (a.act == ALG_ACT_GELU_TANH) {
#pragma unroll
    for (int x = 0; x < 32; ++x) f[x] = gelu_tanh(f[x]);
  }
}
__device__ __forceinline__ void pack_bf16_32(const float (&f)[32], uint32_t (&w)[16]) {
#pragma unroll
  for (int h = 0; h < 16; ++h) {
    __nv_bfloat162 p = __floats2bfloat162_rn(f[2 * h], f[2 * h + 1]);
    w[h] = *(uint32_t *)&p;
  }
}

// Converts one row segment of 32 fp32 accumulator values (bias / activation applied) and stores
// it: 64 bytes of bf16 or 128 bytes of fp32, as 32-byte stores when the address allows.
__device__ __forceinline__ void finish_and_store_32(float (&f)[32], const ProjArgs &a, int64_t out_row, int col) {
  finish_32(f, a, col);
  if (a.y_bf16) {
    uint32_t w[16];
    pack_bf16_32(f, w);
    __nv_bfloat16 *dst = (__nv_bfloat16 *)a.Y + out_row * a.ldy + col;
    if ((((uintptr_t)dst) & 31u) == 0) {  // 32-byte stores fill whole sectors
#pragma unroll
      for (int g = 0; g < 2; ++g)
        asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(dst + g * 16), "r"(w[g * 8]),
                     "r"(w[g * 8 + 1]), "r"(w[g * 8 + 2]), "r"(w[g * 8 + 3]), "r"(w[g * 8 + 4]), "r"(w[g * 8 + 5]),
                     "r"(w[g * 8 + 6]), "r"(w[g * 8 + 7])
                     : "memory");
    } else {
#pragma unroll
      for (int g = 0; g < 4; ++g) ((uint4 *)dst)[g] = make_uint4(w[g * 4], w[g * 4 + 1], w[g * 4 + 2], w[g * 4 + 3]);
    }
  } else {
    float *dst = (float *)a.Y + out_row * a.ldy + col;
    if ((((uintptr_t)dst) & 31u) == 0) {
#pragma unroll
      for (int g = 0; g < 4; ++g)
        asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(dst + g * 8),
                     "r"(__float_as_uint(f[g * 8])), "r"(__float_as_uint(f[g * 8 + 1])),
                     "r"(__float_as_uint(f[g * 8 + 2])), "r"(__float_as_uint(f[g * 8 + 3])),
                     "r"(__float_as_uint(f[g * 8 + 4])), "r"(__float_as_uint(f[g * 8 + 5])),
                     "r"(__float_as_uint(f[g * 8 + 6])), "r"(__float_as_uint(f[g * 8 + 7]))
                     : "memory");
    } else {
#pragma unroll
      for (int g = 0; g < 8; ++g) ((float4 *)dst)[g] = make_float4(f[g * 4], f[g * 4 + 1], f[g * 4 + 2], f[g * 4 + 3]);
    }
  }
}

// Host side: tensor-map encoding through the driver entry point (no link-time libcuda dependency).
cudaError_t make_map_2d(CUtensorMap *map, const void *base, uint64_t inner, uint64_t outer, uint64_t ld_bytes,
                        uint32_t box_inner, uint32_t box_outer);
cudaError_t make_map_2d_sw(CUtensorMap *map, const void *base, uint64_t inner, uint64_t outer, uint64_t ld_bytes,
                           uint32_t box_inner, uint32_t box_outer, int swizzle_bytes);
// General bf16 map of rank 2..5: dims[rank], byte strides of dims 1..rank-1, box[rank], swizzle 128 / 64 / 32 / 0.
cudaError_t make_map_nd(CUtensorMap *map, const void *base, int rank, const uint64_t *dims, const uint64_t *stride_bytes,
                        const uint32_t *box, int swizzle_bytes);
// A operand of either kind: plain rows (2-D) or, for the cyclic schedule, the type-strided view
// {K, q, M/q} of X with strides {ld, q*ld} and a box of 64 x 1 x 128 (same shared-memory image).
cudaError_t make_map_a(CUtensorMap *map, const ProjArgs &a);
cudaError_t make_map_b3d(CUtensorMap *map, const ProjArgs &a, int chunks);

}  // namespace tc
}  // namespace algproj
