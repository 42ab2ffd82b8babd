// Device timeline stamps for kernel tuning.  Everything here is empty unless the library is built
// with -DALGPROJ_TRACE, so default builds carry no tracing code, no extra kernel argument and no
// extra export.
//
// A traced build gives every translation unit that says ALG_TRACE_DEFINE(name) a buffer pointer
// in device memory and an exported setter  alg_trace_set_<name>(void *device_buffer, int cap):
// the buffer holds [slot][cap] int64 records (clock64 << 8 | tag), slot = CTA * 3 + role for the
// first eight CTAs, followed by per-CTA {globaltimer, clock64} pairs at entry and exit (two sets of
// 256 CTAs x 4 slots), followed at slot 24 * cap + 2048 by an append-only log.
#pragma once

#ifdef ALGPROJ_TRACE

#include <cuda_runtime.h>

#define ALG_TRACE_DEFINE(name)                                                              \
  static __device__ long long *alg_trace_buf = nullptr;                                     \
  static __device__ int alg_trace_cap = 0;                                                  \
  extern "C" void alg_trace_set_##name(void *device_buffer, int cap) {                      \
    long long *p = (long long *)device_buffer;                                              \
    cudaMemcpyToSymbol(alg_trace_buf, &p, sizeof(p));                                       \
    cudaMemcpyToSymbol(alg_trace_cap, &cap, sizeof(cap));                                   \
  }
#define ALG_TRACE_VARS [[maybe_unused]] int tr_n = 0
#define ALG_TRACE(role, tag)                                                                        \
  do {                                                                                              \
    if (alg_trace_buf && blockIdx.x < 8 && tr_n < alg_trace_cap)                                    \
      alg_trace_buf[((size_t)blockIdx.x * 3 + (role)) * alg_trace_cap + tr_n++] = (clock64() << 8) | (tag); \
  } while (0)
// whole-CTA window: which = 0 at entry, 1 at exit; `set` (0 or 1) keeps two kernels of a step apart
#define ALG_TRACE_CTA(which, set)                                                                   \
  do {                                                                                              \
    if (alg_trace_buf && threadIdx.x == 0) {                                                        \
      unsigned long long gt_;                                                                       \
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(gt_));                                       \
      long long *w_ = alg_trace_buf + (size_t)24 * alg_trace_cap + (set) * 1024 + blockIdx.x * 4;   \
      w_[(which)] = (long long)gt_;                                                                 \
      w_[2 + (which)] = clock64();                                                                  \
    }                                                                                               \
  } while (0)

// Append-only log shared by all launches: record = {tag, globaltimer, clock64}; the cursor sits at
// buffer slot 24 * cap + 2048, the records follow it.  CTA 0 / thread 0 only.
#define ALG_TRACE_SEQ(tag)                                                                          \
  do {                                                                                              \
    if (alg_trace_buf && blockIdx.x == 0 && threadIdx.x == 0) {                                     \
      long long *base_ = alg_trace_buf + (size_t)24 * alg_trace_cap + 2048;                         \
      const unsigned long long i_ = atomicAdd((unsigned long long *)base_, 1ull);                   \
      if (i_ < 4096) {                                                                              \
        unsigned long long gt_;                                                                     \
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(gt_));                                     \
        base_[1 + 3 * i_] = (tag);                                                                  \
        base_[2 + 3 * i_] = (long long)gt_;                                                         \
        base_[3 + 3 * i_] = clock64();                                                              \
      }                                                                                             \
    }                                                                                               \
  } while (0)

#else

#define ALG_TRACE_SEQ(tag) \
  do {                     \
  } while (0)
#define ALG_TRACE_DEFINE(name)
#define ALG_TRACE_VARS \
  do {                 \
  } while (0)
#define ALG_TRACE(role, tag) \
  do {                       \
  } while (0)
#define ALG_TRACE_CTA(which, set) \
  do {                            \
  } while (0)

#endif
