// Host-side entry to the tensor-core codec kernels.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "ssn_common.cuh"

namespace ssn {

struct MmaArgs {
  const __nv_bfloat16 *src;   // [n x d] rows to project, or nullptr (expand only)
  const __nv_bfloat16 *zin;   // [n x k] coordinates for expand-only
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
                                     int sm_count, cudaStream_t stream);

// mode: 1 = project, 2 = expand, 3 = project then expand (shift must be false).
cudaError_t launch_codec_mma(const MmaArgs &a, bool shift, int mode, int sm_count,
                             cudaStream_t stream);

}  // namespace ssn
