// Shared device helpers of libssn: element types, the per-token shift lookup, status bits.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ssn.h"

namespace ssn {

// ---- element access in fp32 --------------------------------------------------------------
template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) {
  return __bfloat162float(v);
}
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) {
  return __float2bfloat16_rn(v);
}

// ---- the tables both ends of the boundary share (Sec. 4.1) -------------------------------
struct ShiftTables {
  const void *E;      // [vocab x d] or nullptr
  const void *P;      // [max_pos x d] or nullptr
  const int32_t *ids; // [n] (used when E != nullptr)
  const int32_t *pos; // [n] or nullptr: position = t mod seq_len
  int64_t lde, ldp, vocab;
  int32_t max_pos, seq_len;
  int32_t *dev_status; // nullable
  const float *EU;     // [vocab x k] = E U in fp32, or nullptr (compress only)
  const float *PU;     // [max_pos x k] = P U in fp32, or nullptr (compress only)
  int64_t ldeu, ldpu;
};

// Row index into E for token t, or -1 for "no row" (table absent or id out of range, the
// latter also raising the status bit).
__device__ __forceinline__ int64_t embedding_row(const ShiftTables &s, int64_t t) {
  if (s.E == nullptr) return -1;
  int64_t id = s.ids[t];
  if (id < 0 || id >= s.vocab) {
    if (s.dev_status) atomicOr(s.dev_status, SSN_DEV_BAD_ID);
    return -1;
  }
  return id;
}

__device__ __forceinline__ int64_t position_row(const ShiftTables &s, int64_t t) {
  if (s.P == nullptr) return -1;
  int64_t p = s.pos ? (int64_t)s.pos[t] : (t % s.seq_len);
  if (p < 0 || p >= s.max_pos) {
    if (s.dev_status) atomicOr(s.dev_status, SSN_DEV_BAD_POS);
    return -1;
  }
  return p;
}

}  // namespace ssn
