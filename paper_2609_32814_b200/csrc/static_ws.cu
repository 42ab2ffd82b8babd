// alg_proj_forward_static: the projection forward pass for callers that must not allocate
// device memory.  The scratch that alg_proj_forward takes as a caller-provided workspace lives
// here in a fixed array inside the library image, so the call itself needs no cudaMalloc, no
// cudaFree and no allocator of any framework.
#include "common.cuh"

namespace {

// Scratch of every alg_proj_forward_static call on a device: row permutation, bucket offsets
// and the type-bucketed copy of X.  Each GPU that loads the library holds these
// 8 MiB until the process exits.
constexpr size_t kStaticScratchBytes = ALG_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
void *g_scratch_addr[kMaxDevices] = {nullptr};

// The array's name is only a host-side stand-in; kernels need its device address, which is
// looked up once per device with that device current.
// `handle_dev`: the device the handle's tables live on; the array of any other device is useless
// to it, so a call with another device current is refused.
alg_status_t scratch_address(int handle_dev, void **out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return ALG_ERR_CUDA;
  if (dev != handle_dev) return ALG_ERR_INVALID_ARG;
  if (dev < 0 || dev >= kMaxDevices) return ALG_ERR_UNSUPPORTED_SHAPE;
  if (!g_scratch_addr[dev]) {
    void *p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return ALG_ERR_CUDA;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return ALG_OK;
}

}  // namespace

extern "C" alg_status_t alg_proj_forward_static(alg_proj_t h, const void *X, int64_t ldx, const int32_t *types,
                                                int64_t M, const void *W, int64_t ldw, const void *bias,
                                                alg_act_t act, void *Y, int64_t ldy, alg_dtype_t y_dtype,
                                                void *stream) {
  if (!h || M < 0) return ALG_ERR_INVALID_ARG;
  size_t need = 0;
  alg_status_t s = alg_proj_workspace_bytes(h, M, &need);
  if (s != ALG_OK) return s;
  if (need > kStaticScratchBytes) return ALG_ERR_WORKSPACE_TOO_SMALL;  // problem exceeds the built-in scratch
  void *scratch = nullptr;
  s = scratch_address(algproj::handle_device(h), &scratch);
  if (s != ALG_OK) return s;
  return alg_proj_forward(h, X, ldx, types, M, W, ldw, bias, act, Y, ldy, y_dtype, scratch, kStaticScratchBytes,
                          stream);
}
