// General kernels of libssn: any element type, any rank, any leading dimension or alignment.
// They are the fp32 path and the fallback for shapes the tensor-core kernels do not take.
// Plain fp32 FMAs; one warp owns one token (or one row of W) and reduces over d with shuffles.
#pragma once

#include "ssn_common.cuh"

namespace ssn {

struct TokenArgs {
  const void *src;   // [n x d] rows to project (X, G or W), or nullptr: read coordinates from zin
  const void *src2;  // [n x d] second addend of the rows to project (projection only), or nullptr
  int64_t lds2;
  const void *zin;   // [n x k] coordinates when src == nullptr
  void *zout;        // [n x k] coordinates out, nullable
  void *dst;         // [n x d] expansion out, nullable (may alias src row-for-row)
  const void *U;
  int64_t lds, ldzin, ldzout, lddst, ldu;
  int64_t n;
  int32_t d, k;
  const void *U2;     // expansion factor [d2 x k] when it differs from U (Eq. reparam), else nullptr
  int64_t ldu2;
  int32_t d2;
  // wire rows (the bandwidth estimate of Sec. 3.5 counts the boundary tensors in FP32): the
  // coordinates leave (zout, when projecting) or arrive (zin, when expanding) as fp32 words,
  // leading dimension in words; with wire_ids word k of an outgoing row is the token id
  int32_t wire, wire_ids;
  float *rowsumsq;    // [n] sum of squares of the fp32 output row (before rounding), or nullptr
  int32_t sub_shift;  // phase 1 subtracts E[ids]+P[pos]   (Eq. ssn_compress)
  int32_t add_shift;  // phase 2 adds E[ids]+P[pos] back   (receiver side)
  ShiftTables shift;
};

constexpr int kGenericWarps = 8;
constexpr int kGenericKChunk = 8;

template <typename T>
__global__ void __launch_bounds__(kGenericWarps * 32)
token_kernel(const TokenArgs a) {
  extern __shared__ float zs_all[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t t = (int64_t)blockIdx.x * kGenericWarps + warp;
  if (t >= a.n) return;
  float *zs = zs_all + (size_t)warp * a.k;
  const T *U = static_cast<const T *>(a.U);

  const T *erow = nullptr, *prow = nullptr;
  if (a.sub_shift || a.add_shift) {
    int64_t er = embedding_row(a.shift, t), pr = position_row(a.shift, t);
    if (er >= 0) erow = static_cast<const T *>(a.shift.E) + er * a.shift.lde;
    if (pr >= 0) prow = static_cast<const T *>(a.shift.P) + pr * a.shift.ldp;
  }

  if (a.src != nullptr) {
    const T *x = static_cast<const T *>(a.src) + t * a.lds;
    const T *x2 = a.src2 != nullptr ? static_cast<const T *>(a.src2) + t * a.lds2 : nullptr;
    for (int j0 = 0; j0 < a.k; j0 += kGenericKChunk) {
      float acc[kGenericKChunk];
#pragma unroll
      for (int jj = 0; jj < kGenericKChunk; ++jj) acc[jj] = 0.f;
      const int jn = min(kGenericKChunk, a.k - j0);
      for (int i = lane; i < a.d; i += 32) {
        float r = to_f32(x[i]);
        if (x2 != nullptr) r += to_f32(x2[i]);
        if (a.sub_shift) {
          if (erow) r -= to_f32(erow[i]);
          if (prow) r -= to_f32(prow[i]);
        }
        const T *urow = U + (int64_t)i * a.ldu + j0;
#pragma unroll
        for (int jj = 0; jj < kGenericKChunk; ++jj)
          if (jj < jn) acc[jj] = fmaf(r, to_f32(urow[jj]), acc[jj]);
      }
#pragma unroll
      for (int jj = 0; jj < kGenericKChunk; ++jj) {
        float v = acc[jj];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
        if (lane == 0 && jj < jn) zs[j0 + jj] = v;
      }
    }
    __syncwarp();
    if (a.zout != nullptr && a.wire) {
      float *z = static_cast<float *>(a.zout) + t * a.ldzout;
      for (int j = lane; j < a.k; j += 32) z[j] = zs[j];
      if (a.wire_ids && lane == 0) reinterpret_cast<int32_t *>(z)[a.k] = a.shift.ids[t];
    } else if (a.zout != nullptr) {
      T *z = static_cast<T *>(a.zout) + t * a.ldzout;
      for (int j = lane; j < a.k; j += 32) z[j] = from_f32<T>(zs[j]);
    }
  } else if (a.wire) {
    const float *z = static_cast<const float *>(a.zin) + t * a.ldzin;
    for (int j = lane; j < a.k; j += 32) zs[j] = z[j];
    __syncwarp();
  } else {
    const T *z = static_cast<const T *>(a.zin) + t * a.ldzin;
    for (int j = lane; j < a.k; j += 32) zs[j] = to_f32(z[j]);
    __syncwarp();
  }

  if (a.dst != nullptr) {
    T *out = static_cast<T *>(a.dst) + t * a.lddst;
    const T *Ux = a.U2 != nullptr ? static_cast<const T *>(a.U2) : U;
    const int64_t ldux = a.U2 != nullptr ? a.ldu2 : a.ldu;
    const int dx = a.U2 != nullptr ? a.d2 : a.d;
    float ss = 0.f;
    for (int i = lane; i < dx; i += 32) {
      const T *urow = Ux + (int64_t)i * ldux;
      float acc = 0.f;
      for (int j = 0; j < a.k; ++j) acc = fmaf(zs[j], to_f32(urow[j]), acc);
      if (a.add_shift) {
        if (erow) acc += to_f32(erow[i]);
        if (prow) acc += to_f32(prow[i]);
      }
      ss = fmaf(acc, acc, ss);
      out[i] = from_f32<T>(acc);
    }
    if (a.rowsumsq != nullptr) {
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
      if (lane == 0) a.rowsumsq[t] = ss;
    }
  }
}

// ---- row gather: out[t, 0:kpad] = table[ids[t], 0:k] (zeros past k and for ids outside) -----
struct GatherArgs {
  const void *table;
  void *out;
  const int32_t *ids;
  int64_t ld_table, ld_out, n, rows;
  int32_t k, kpad;
  int32_t *dev_status;   // nullable: SSN_DEV_BAD_ID when an id is outside [0, rows)
};

template <typename T>
__global__ void gather_rows_kernel(const GatherArgs a) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= a.n * a.kpad) return;
  const int64_t t = i / a.kpad;
  const int j = (int)(i - t * a.kpad);
  const int64_t id = a.ids[t];
  T v = from_f32<T>(0.f);
  const bool in_table = id >= 0 && id < a.rows;
  if (j < a.k && in_table) v = static_cast<const T *>(a.table)[id * a.ld_table + j];
  if (!in_table && j == 0 && a.dev_status) atomicOr(a.dev_status, SSN_DEV_BAD_ID);
  static_cast<T *>(a.out)[t * a.ld_out + j] = v;
}

// The same with blocks of (kpad x rows) threads, thread (j, y) = column j of one row: no index
// division (kpad <= 256).
template <typename T>
__global__ void gather_rows_2d_kernel(const GatherArgs a) {
  const int64_t t = (int64_t)blockIdx.x * blockDim.y + threadIdx.y;
  const int j = threadIdx.x;
  if (t >= a.n) return;
  const int64_t id = a.ids[t];
  T v = from_f32<T>(0.f);
  const bool in_table = id >= 0 && id < a.rows;
  if (j < a.k && in_table) v = static_cast<const T *>(a.table)[id * a.ld_table + j];
  if (!in_table && j == 0 && a.dev_status) atomicOr(a.dev_status, SSN_DEV_BAD_ID);
  static_cast<T *>(a.out)[t * a.ld_out + j] = v;
}

// ---- wire rows in: ids out of word k, coordinates as bf16 head + remainder; the basis twice -----
// One launch prepares both operands of the split expansion.  Blocks are (kp x rows_per_block)
// threads: thread (j, y) owns column j of one row, so nothing is divided.
//   blocks [0, split_blocks):  row t of the wire buffer -> ids[t] (word k) and, when split is given,
//       split[t] = (head | remainder) in columns [0, k) and [kp, kp + k), zeros elsewhere
//   blocks [split_blocks, ..): row r of U -> U2[r] = (U[r] 0 | U[r] 0), so that
//       (head | remainder) U2^T = (head + remainder) U^T
struct WirePrepareArgs {
  const float *wire;        // [n x ldw] words
  __nv_bfloat16 *split;     // [n x 2 kp] or nullptr
  int32_t *ids;             // [n] or nullptr
  const __nv_bfloat16 *U;   // [d x k], leading dimension ldu (split only)
  __nv_bfloat16 *U2;        // [d x 2 kp] (split only)
  int64_t ldw, ldu, n;
  int32_t k, kp, d;
  int32_t split_blocks;
};

static __global__ void wire_prepare_kernel(const WirePrepareArgs a) {
  const int j = threadIdx.x;
  if ((int)blockIdx.x < a.split_blocks) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.y + threadIdx.y;
    if (t >= a.n) return;
    const float *row = a.wire + t * a.ldw;
    if (a.ids != nullptr && j == 0) a.ids[t] = reinterpret_cast<const int32_t *>(row)[a.k];
    if (a.split != nullptr) {
      const float z = j < a.k ? row[j] : 0.f;
      const __nv_bfloat16 head = __float2bfloat16_rn(z);
      a.split[t * 2 * a.kp + j] = head;
      a.split[t * 2 * a.kp + a.kp + j] = __float2bfloat16_rn(z - __bfloat162float(head));
    }
  } else {
    const int64_t r = (int64_t)(blockIdx.x - a.split_blocks) * blockDim.y + threadIdx.y;
    if (r >= a.d) return;
    const __nv_bfloat16 v = j < a.k ? a.U[r * a.ldu + j] : __float2bfloat16_rn(0.f);
    a.U2[r * 2 * a.kp + j] = v;
    a.U2[r * 2 * a.kp + a.kp + j] = v;
  }
}

// ---- contraction over tokens: out [m x k] (fp32) = H^T C, H [n x m], C [n x k] ---------------
struct TokensContractArgs {
  const void *H, *C;
  float *out;
  int64_t ldh, ldc, ldout, n;
  int32_t m, k;
};

// One thread per output element, 32 rows x 8 columns per block; the loads of H are coalesced.
template <typename T>
__global__ void __launch_bounds__(256) tokens_contract_kernel(const TokensContractArgs a) {
  const int r = blockIdx.x * 32 + (threadIdx.x & 31), j = blockIdx.y * 8 + (threadIdx.x >> 5);
  if (r >= a.m || j >= a.k) return;
  const T *H = static_cast<const T *>(a.H), *C = static_cast<const T *>(a.C);
  float acc = 0.f;
  for (int64_t t = 0; t < a.n; ++t) acc = fmaf(to_f32(H[t * a.ldh + r]), to_f32(C[t * a.ldc + j]), acc);
  a.out[(int64_t)r * a.ldout + j] = acc;
}

// ---- prepared tables: out [n x k] (fp32) = rows_in [n x d] U --------------------------------
struct TableArgs {
  const void *rows_in;   // E or P
  const void *U;
  float *out;
  int64_t ld_in, ldu, ld_out, n;
  int32_t d, k;
};

constexpr int kTableWarps = 8;

// One warp per row; the lanes split d and reduce with shuffles, 8 columns of U at a time.
template <typename T>
__global__ void __launch_bounds__(kTableWarps * 32) table_project_kernel(const TableArgs a) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t t = (int64_t)blockIdx.x * kTableWarps + warp;
  if (t >= a.n) return;
  const T *row = static_cast<const T *>(a.rows_in) + t * a.ld_in;
  const T *U = static_cast<const T *>(a.U);
  for (int j0 = 0; j0 < a.k; j0 += kGenericKChunk) {
    const int jn = min(kGenericKChunk, a.k - j0);
    float acc[kGenericKChunk];
#pragma unroll
    for (int jj = 0; jj < kGenericKChunk; ++jj) acc[jj] = 0.f;
    for (int i = lane; i < a.d; i += 32) {
      const float r = to_f32(row[i]);
      const T *urow = U + (int64_t)i * a.ldu + j0;
#pragma unroll
      for (int jj = 0; jj < kGenericKChunk; ++jj)
        if (jj < jn) acc[jj] = fmaf(r, to_f32(urow[jj]), acc[jj]);
    }
#pragma unroll
    for (int jj = 0; jj < kGenericKChunk; ++jj) {
      float v = acc[jj];
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
      if (lane == 0 && jj < jn) a.out[t * a.ld_out + j0 + jj] = v;
    }
  }
}

// ---- LEFT re-projection, W [d x m]:  T = U^T W  then  W = U T ------------------------------
struct LeftArgs {
  void *W;          // [d x m]
  const void *U;    // [d x k]
  float *T;         // [k x m] fp32 scratch
  int64_t ldw, ldu, m;
  int32_t d, k;
};

constexpr int kLeftCols = 128;

// T[j][c] = sum_i U[i][j] W[i][c]; thread = column c, blockIdx.y = chunk of 8 coordinates.
template <typename T>
__global__ void __launch_bounds__(kLeftCols) left_reduce_kernel(const LeftArgs a) {
  const int64_t c = (int64_t)blockIdx.x * kLeftCols + threadIdx.x;
  const int j0 = blockIdx.y * kGenericKChunk;
  const int jn = min(kGenericKChunk, a.k - j0);
  if (c >= a.m) return;
  const T *W = static_cast<const T *>(a.W);
  const T *U = static_cast<const T *>(a.U);
  float acc[kGenericKChunk];
#pragma unroll
  for (int jj = 0; jj < kGenericKChunk; ++jj) acc[jj] = 0.f;
  for (int i = 0; i < a.d; ++i) {
    const float w = to_f32(W[(int64_t)i * a.ldw + c]);
    const T *urow = U + (int64_t)i * a.ldu + j0;
#pragma unroll
    for (int jj = 0; jj < kGenericKChunk; ++jj)
      if (jj < jn) acc[jj] = fmaf(to_f32(urow[jj]), w, acc[jj]);
  }
#pragma unroll
  for (int jj = 0; jj < kGenericKChunk; ++jj)
    if (jj < jn) a.T[(int64_t)(j0 + jj) * a.m + c] = acc[jj];
}

// W[i][c] = sum_j U[i][j] T[j][c]; thread = column c, blockIdx.y = block of 32 rows.
template <typename T>
__global__ void __launch_bounds__(kLeftCols) left_expand_kernel(const LeftArgs a) {
  const int64_t c = (int64_t)blockIdx.x * kLeftCols + threadIdx.x;
  if (c >= a.m) return;
  T *W = static_cast<T *>(a.W);
  const T *U = static_cast<const T *>(a.U);
  const int i0 = blockIdx.y * 32, i1 = min(a.d, i0 + 32);
  for (int i = i0; i < i1; ++i) {
    const T *urow = U + (int64_t)i * a.ldu;
    float acc = 0.f;
    for (int j = 0; j < a.k; ++j) acc = fmaf(to_f32(urow[j]), a.T[(int64_t)j * a.m + c], acc);
    W[(int64_t)i * a.ldw + c] = from_f32<T>(acc);
  }
}

}  // namespace ssn
