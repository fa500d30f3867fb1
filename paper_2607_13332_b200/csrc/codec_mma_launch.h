// Host-side entry to the tensor-core codec kernels.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <atomic>

#include "ssn_common.cuh"

namespace ssn {

struct MmaArgs {
  const __nv_bfloat16 *src;   // [n x d] rows to project, or nullptr (expand only)
  const __nv_bfloat16 *zin;   // [n x k] coordinates for expand-only
  // tcgen05 expansion only, k <= 64: a second [n x k] coordinate matrix (same leading dimension)
  // whose product with U^T is added to the first one's (the bf16 remainder of fp32 wire rows); nullptr: none
  const __nv_bfloat16 *zin2;
  __nv_bfloat16 *zout;        // [n x k] coordinates out, nullable
  __nv_bfloat16 *dst;         // [n x d] expansion out, nullable
  const __nv_bfloat16 *U;     // [d x k], 16-byte aligned, ldu % 8 == 0
  int64_t lds, ldzin, ldzout, lddst, ldu;
  int64_t n;
  int32_t d, k;
  int32_t pshare;             // projection kernel: the batch is whole sequences, share P U per block
  // project-then-expand with two different factors (Eq. reparam, Y = (H Z) U^T): the rows of src
  // have d1 columns and are contracted with B1 [d1 x k]; nullptr: B1 = U, d1 = d
  const __nv_bfloat16 *B1;
  int64_t ldb1;
  int32_t d1;
  // projection of a sum (the stage's last residual add fused into compress): Z = (src + src2) U,
  // tcgen05 projection without row operands only; nullptr: none
  const __nv_bfloat16 *src2;
  int64_t lds2;
  // projection with wire rows: the coordinates are stored as fp32 words in zout32 (zout is
  // nullptr then); wire_ids != nullptr: word k of row t is wire_ids[t]
  float *zout32;
  int64_t ldzout32;
  const int32_t *wire_ids;
  // expansion with the row statistic: rowsumsq[t] += sum of squares of the fp32 output row t
  // (zeroed by the caller); only the tcgen05 expansion takes it
  float *rowsumsq;
  ShiftTables shift;
};

// Shapes the tensor-core kernels take (alignment is checked by the caller).
bool codec_mma_supports(int d, int k);

// Most matrices one launch of the fused project-then-expand kernel takes (its tensor maps travel
// as kernel parameters: 2 x 128 bytes per matrix).
constexpr int kMaxFusedMatrices = 32;

// Project-then-expand of up to kMaxFusedMatrices matrices in ONE launch of the tcgen05 kernel (a.U, a.ldu, a.d,
// a.k are read from `a`): [rows[i] x d] with the subspace on the columns, or, with `left`,
// [d x rows[i]] with the subspace on the rows.  cudaErrorNotSupported when the shapes or
// alignments are not the kernel's, and nothing has been launched then.
cudaError_t launch_codec_umma_roundtrip_list(const MmaArgs &a, const __nv_bfloat16 *const *src,
                                             __nv_bfloat16 *const *dst, const int64_t *rows,
                                             const int64_t *lds, const int64_t *lddst, int count,
                                             int sm_count, cudaStream_t stream, bool left);

// out [m x k] (fp32) = H^T C on tcgen05 (H: [n x m], C: [n x k], both bf16); cudaErrorNotSupported
// when the shapes or alignments are not the kernel's, and nothing has been launched then.  The
// output is zeroed on the stream first when several CTAs share a row block.
cudaError_t launch_codec_umma_tokens(const __nv_bfloat16 *H, int64_t ldh, const __nv_bfloat16 *C, int64_t ldc,
                                     float *out, int64_t ldout, int64_t n, int32_t m, int32_t k,
                                     int32_t *dev_status, int sm_count, cudaStream_t stream);

// The self-test of the bounded waits (see ssn_selftest_bounded_wait).
cudaError_t launch_bounded_wait_selftest(int max_polls, int32_t *dev_status, cudaStream_t stream);

// Adds to the process-wide launch counter behind ssn_launch_count().
void count_launches(int launches);

// Records the kernel a launch used for ssn_last_kernel(): an SSN_KERNEL_* family and SSN_KVAR_* bits.
void note_kernel(int family, int variant);

// cudaFuncAttributeMaxDynamicSharedMemorySize belongs to the current device's context: it is set
// once per device (`done` holds one bit per device ordinal) and always for ordinals past 63.
template <typename Kernel>
cudaError_t allow_dynamic_smem(Kernel kernel, int smem, std::atomic<uint64_t> &done) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const uint64_t bit = dev >= 0 && dev < 64 ? 1ull << dev : 0ull;
  if (bit != 0 && (done.load(std::memory_order_acquire) & bit)) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e == cudaSuccess && bit != 0) done.fetch_or(bit, std::memory_order_release);
  return e;
}

// Launch of a tcgen05 kernel that may START before the kernel in front of it in the stream has
// ended (programmatic dependent launch): its CTAs set up their barriers and tensor memory on the SMs
// the earlier kernel has left, and wait (griddepcontrol.wait, which every such kernel executes after
// its set-up and before it touches global memory) until that kernel is complete and its writes are
// visible.  The earlier kernel allows this at its start (griddepcontrol.launch_dependents); behind
// any other kernel, and inside a stream capture, the launch is an ordinary one.  cluster = 2 launches
// pairs of CTAs.
template <typename Kernel, typename... Args>
cudaError_t launch_dependent(Kernel kernel, unsigned grid, int threads, int smem, cudaStream_t stream, int cluster,
                             Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3((unsigned)threads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  int n = 0;
  if (cluster > 1) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = (unsigned)cluster;
    attr[n].val.clusterDim.y = 1;
    attr[n].val.clusterDim.z = 1;
    ++n;
  }
  cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(stream, &capturing) == cudaSuccess && capturing == cudaStreamCaptureStatusNone) {
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}

// The tcgen05 kernels one by one; each returns cudaErrorNotSupported, with nothing launched, for
// shapes and alignments that are not its own (the conditions are stated at the definitions).
cudaError_t launch_codec_umma_project(const MmaArgs &a, bool shift, int sm_count, cudaStream_t stream);
cudaError_t launch_codec_umma_expand(const MmaArgs &a, bool shift, int sm_count, cudaStream_t stream);
cudaError_t launch_codec_umma_roundtrip(const MmaArgs &a, int sm_count, cudaStream_t stream);

// mode: 1 = project, 2 = expand, 3 = project then expand (shift must be false).
cudaError_t launch_codec_mma(const MmaArgs &a, bool shift, int mode, int sm_count,
                             cudaStream_t stream);

}  // namespace ssn
