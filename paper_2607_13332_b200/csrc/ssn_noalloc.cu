// ssn_weight_reproject_left_static: the LEFT re-projection with its scratch in a fixed device
// array owned by the library, for callers that cannot provide (or allocate) a workspace.
#include "ssn.h"

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <atomic>

#include "codec_mma_launch.h"
#include "generic_kernels.cuh"

namespace ssn {
namespace {

// The k x m coordinates T = U^T W live here between the two kernels.  Every GPU that loads the
// library holds these 4 MiB until the process exits.
constexpr size_t kStaticScratchBytes = SSN_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::atomic<float *> g_scratch_ptr[kMaxDevices];   // device address of g_static_scratch, per device (0 = not set up)

// The array's name is only a host-side handle; kernels need its device address, which the
// runtime hands out per device (the device that is current when it is asked).
float *scratch_of_current_device() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    cudaGetLastError();
    return nullptr;
  }
  float *known = g_scratch_ptr[dev].load(std::memory_order_acquire);
  if (known == nullptr) {   // two threads may both ask; they get the same address
    void *p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) {
      cudaGetLastError();
      return nullptr;
    }
    known = static_cast<float *>(p);
    g_scratch_ptr[dev].store(known, std::memory_order_release);
  }
  return known;
}

}  // namespace
}  // namespace ssn

using namespace ssn;

extern "C" {

size_t ssn_static_scratch_bytes(void) { return kStaticScratchBytes; }

ssn_status_t ssn_weight_reproject_left_static(const ssn_codec_t *codec, void *W, int64_t cols,
                                              int64_t ldw, void *stream) {
  if (codec == nullptr || codec->U == nullptr) return SSN_ERR_NULL;
  if (codec->dtype != SSN_F32 && codec->dtype != SSN_BF16) return SSN_ERR_DTYPE;
  if (codec->d < 1 || codec->k < 1 || codec->k > codec->d || codec->ldu < codec->k) return SSN_ERR_SHAPE;
  if (cols < 1 || ldw < cols) return SSN_ERR_SHAPE;
  if (W == nullptr) return SSN_ERR_NULL;
  // the fixed scratch must hold k x cols fp32 coordinates
  if ((size_t)codec->k * (size_t)cols > kStaticScratchBytes / sizeof(float)) return SSN_ERR_WORKSPACE;
  const int64_t col_blocks = (cols + kLeftCols - 1) / kLeftCols;
  // both kernels' grids must be launchable before the first one runs
  if (col_blocks > 0x7fffffffLL || ((int64_t)codec->d + 31) / 32 > 65535) return SSN_ERR_SHAPE;
  float *scratch = scratch_of_current_device();
  if (scratch == nullptr) return SSN_ERR_CUDA;

  LeftArgs a{};
  a.W = W;
  a.U = codec->U;
  a.T = scratch;   // fully rewritten by the first kernel: nothing of the last call survives
  a.ldw = ldw;
  a.ldu = codec->ldu;
  a.m = cols;
  a.d = codec->d;
  a.k = codec->k;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  dim3 g1((unsigned)col_blocks, (unsigned)((codec->k + kGenericKChunk - 1) / kGenericKChunk));
  dim3 g2((unsigned)col_blocks, (unsigned)((codec->d + 31) / 32));
  if (codec->dtype == SSN_F32) {
    left_reduce_kernel<float><<<g1, kLeftCols, 0, s>>>(a);
    left_expand_kernel<float><<<g2, kLeftCols, 0, s>>>(a);
  } else {
    left_reduce_kernel<__nv_bfloat16><<<g1, kLeftCols, 0, s>>>(a);
    left_expand_kernel<__nv_bfloat16><<<g2, kLeftCols, 0, s>>>(a);
  }
  count_launches(2);
  note_kernel(SSN_KERNEL_GENERIC, 0);
  return cudaGetLastError() == cudaSuccess ? SSN_OK : SSN_ERR_CUDA;
}

}  // extern "C"
