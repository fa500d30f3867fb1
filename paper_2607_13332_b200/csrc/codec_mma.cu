// Instantiations and launcher of the tensor-core codec kernels (see codec_mma.cuh).
#include "codec_mma.cuh"


#include "codec_mma_launch.h"

namespace ssn {
namespace {

template <int NT, int MT, bool SHIFT, int MODE>
cudaError_t launch_one(const MmaArgs &a, int sm_count, cudaStream_t stream) {
  auto kernel = codec_mma_kernel<NT, MT, SHIFT, MODE>;
  constexpr int smem = kStages * UStageRing<NT>::kStageBytes;
  static bool configured = false;   // per instantiation; the attribute is per-context state
  if (smem > 48 * 1024 && !configured) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  int64_t grid = (a.n + 15) / 16;
  if (grid > sm_count) grid = sm_count;
  kernel<<<(unsigned)grid, kMmaThreads, smem, stream>>>(a);
  return cudaGetLastError();
}

template <int NT, int MT>
cudaError_t launch_nt(const MmaArgs &a, bool shift, int mode, int sm_count, cudaStream_t s) {
  if (mode == kModeProject)
    return shift ? launch_one<NT, MT, true, kModeProject>(a, sm_count, s)
                 : launch_one<NT, MT, false, kModeProject>(a, sm_count, s);
  if (mode == kModeExpand)
    return shift ? launch_one<NT, MT, true, kModeExpand>(a, sm_count, s)
                 : launch_one<NT, MT, false, kModeExpand>(a, sm_count, s);
  return launch_one<NT, MT, false, kModeBoth>(a, sm_count, s);
}

}  // namespace

bool codec_mma_supports(int d, int k) {
  return d % 32 == 0 && (int64_t)d * 2 <= kZeroRowBytes && k >= 1 && k <= 128;
}

cudaError_t launch_codec_mma(const MmaArgs &a, bool shift, int mode, int sm_count,
                             cudaStream_t stream) {
  const int nt = (a.k + 7) / 8;
  // With few tokens per warp a second 16-row tile would be computed for nothing.
  const bool small = a.n <= (int64_t)sm_count * kMmaWarps * 16;
  if (small) {
    if (nt <= 1) return launch_nt<1, 1>(a, shift, mode, sm_count, stream);
    if (nt <= 2) return launch_nt<2, 1>(a, shift, mode, sm_count, stream);
    if (nt <= 4) return launch_nt<4, 1>(a, shift, mode, sm_count, stream);
    if (nt <= 5) return launch_nt<5, 1>(a, shift, mode, sm_count, stream);
    if (nt <= 6) return launch_nt<6, 1>(a, shift, mode, sm_count, stream);
    if (nt <= 8) return launch_nt<8, 1>(a, shift, mode, sm_count, stream);
  } else {
    if (nt <= 1) return launch_nt<1, 2>(a, shift, mode, sm_count, stream);
    if (nt <= 2) return launch_nt<2, 2>(a, shift, mode, sm_count, stream);
    if (nt <= 4) return launch_nt<4, 2>(a, shift, mode, sm_count, stream);
    if (nt <= 5) return launch_nt<5, 2>(a, shift, mode, sm_count, stream);
    if (nt <= 6) return launch_nt<6, 2>(a, shift, mode, sm_count, stream);
    if (nt <= 8) return launch_nt<8, 2>(a, shift, mode, sm_count, stream);
  }
  if (nt <= 12) return launch_nt<12, 1>(a, shift, mode, sm_count, stream);
  return launch_nt<16, 1>(a, shift, mode, sm_count, stream);
}

}  // namespace ssn
