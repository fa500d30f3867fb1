// General kernels of libssn: any element type, any rank, any leading dimension or alignment.
// They are the fp32 path and the fallback for shapes the tensor-core kernels do not take.
// Plain fp32 FMAs; a warp owns two tokens (or rows of W), U is staged through shared memory.
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
constexpr int kGenericKChunk = 8;     // coordinates per pass of the table and LEFT kernels below
constexpr int kGenericTokens = 2;     // tokens per warp
constexpr int kGenericCoords = 32;    // coordinates per pass
constexpr int kGenericRows = 64;      // rows of U staged in shared memory at a time (two per lane)
constexpr int kGenericTokensPerBlock = kGenericWarps * kGenericTokens;

// Dynamic shared memory: the coordinates of the block's tokens (fp32) and one staged piece of U.
inline size_t generic_token_smem_bytes(int k) {
  return ((size_t)kGenericTokensPerBlock * k + (size_t)kGenericRows * (kGenericCoords + 1)) * sizeof(float);
}

// A warp owns kGenericTokens tokens; its lanes split d.  U is staged through shared memory in
// pieces of kGenericRows rows x kGenericCoords coordinates (fp32, row pitch odd, so that the lanes,
// which read different rows, hit different banks) by all warps of the block together, and every
// staged value is used for both tokens of every warp.
//   projection: lane l holds rows l and l + 32 of the piece: r = x - e - p for both tokens, then
//       acc[token][coordinate] += r * U[row][coordinate] for the 32 coordinates of the pass;
//       shuffle reduction over the lanes at the end of a pass.  The row is re-read once per pass.
//   expansion: lane l produces columns l and l + 32 of the piece: acc[token][column] +=
//       z[token][coordinate] * U[column][coordinate] over all passes, then the shift terms are
//       added and the row statistic (if asked for) is summed before the rounding.
template <typename T>
__global__ void __launch_bounds__(kGenericWarps * 32)
token_kernel(const TokenArgs a) {
  extern __shared__ float smem_f[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float *zs = smem_f + (size_t)warp * kGenericTokens * a.k;               // [token][k] of this warp
  float *us = smem_f + (size_t)kGenericTokensPerBlock * a.k;              // [kGenericRows][kGenericCoords + 1]
  constexpr int kPitch = kGenericCoords + 1;
  const int64_t t0 = ((int64_t)blockIdx.x * kGenericWarps + warp) * kGenericTokens;
  const T *U = static_cast<const T *>(a.U);

  bool valid[kGenericTokens];
  const T *erow[kGenericTokens], *prow[kGenericTokens];
#pragma unroll
  for (int tk = 0; tk < kGenericTokens; ++tk) {
    valid[tk] = t0 + tk < a.n;
    erow[tk] = prow[tk] = nullptr;
    if (valid[tk] && (a.sub_shift || a.add_shift)) {
      const int64_t er = embedding_row(a.shift, t0 + tk), pr = position_row(a.shift, t0 + tk);
      if (er >= 0) erow[tk] = static_cast<const T *>(a.shift.E) + er * a.shift.lde;
      if (pr >= 0) prow[tk] = static_cast<const T *>(a.shift.P) + pr * a.shift.ldp;
    }
  }
  // stages rows [i0, i0 + kGenericRows) x coordinates [j0, j0 + kGenericCoords) of `src` (zeros outside)
  auto stage_u = [&](const T *src, int64_t ld, int rows, int i0, int j0) {
    __syncthreads();   // the previous piece has been read by everyone
    for (int e = threadIdx.x; e < kGenericRows * kGenericCoords; e += kGenericWarps * 32) {
      const int ii = e / kGenericCoords, jj = e % kGenericCoords;
      const int i = i0 + ii, j = j0 + jj;
      us[ii * kPitch + jj] = (i < rows && j < a.k) ? to_f32(src[(int64_t)i * ld + j]) : 0.f;
    }
    __syncthreads();
  };

  if (a.src != nullptr) {
    const T *x[kGenericTokens], *x2[kGenericTokens];
#pragma unroll
    for (int tk = 0; tk < kGenericTokens; ++tk) {
      x[tk] = static_cast<const T *>(a.src) + (valid[tk] ? t0 + tk : 0) * a.lds;
      x2[tk] = a.src2 != nullptr ? static_cast<const T *>(a.src2) + (valid[tk] ? t0 + tk : 0) * a.lds2 : nullptr;
    }
    for (int j0 = 0; j0 < a.k; j0 += kGenericCoords) {
      float acc[kGenericTokens][kGenericCoords];
#pragma unroll
      for (int tk = 0; tk < kGenericTokens; ++tk)
#pragma unroll
        for (int jj = 0; jj < kGenericCoords; ++jj) acc[tk][jj] = 0.f;
      for (int i0 = 0; i0 < a.d; i0 += kGenericRows) {
        // the residuals of this piece first: their loads are in flight while U is being staged
        float r[kGenericRows / 32][kGenericTokens];
#pragma unroll
        for (int h = 0; h < kGenericRows / 32; ++h) {
          const int i = i0 + lane + 32 * h;
#pragma unroll
          for (int tk = 0; tk < kGenericTokens; ++tk) {
            float v = 0.f;
            if (valid[tk] && i < a.d) {
              v = to_f32(x[tk][i]);
              if (x2[tk] != nullptr) v += to_f32(x2[tk][i]);
              if (a.sub_shift) {
                if (erow[tk]) v -= to_f32(erow[tk][i]);
                if (prow[tk]) v -= to_f32(prow[tk][i]);
              }
            }
            r[h][tk] = v;
          }
        }
        stage_u(U, a.ldu, a.d, i0, j0);
#pragma unroll
        for (int h = 0; h < kGenericRows / 32; ++h) {
          const float *urow = us + (lane + 32 * h) * kPitch;
#pragma unroll
          for (int jj = 0; jj < kGenericCoords; ++jj) {
            const float u = urow[jj];
#pragma unroll
            for (int tk = 0; tk < kGenericTokens; ++tk) acc[tk][jj] = fmaf(r[h][tk], u, acc[tk][jj]);
          }
        }
      }
#pragma unroll
      for (int tk = 0; tk < kGenericTokens; ++tk)
#pragma unroll
        for (int jj = 0; jj < kGenericCoords; ++jj) {
          float v = acc[tk][jj];
#pragma unroll
          for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
          if (lane == 0 && j0 + jj < a.k) zs[tk * a.k + j0 + jj] = v;
        }
    }
    __syncwarp();
#pragma unroll
    for (int tk = 0; tk < kGenericTokens; ++tk) {
      if (!valid[tk] || a.zout == nullptr) continue;
      const int64_t t = t0 + tk;
      if (a.wire) {
        float *z = static_cast<float *>(a.zout) + t * a.ldzout;
        for (int j = lane; j < a.k; j += 32) z[j] = zs[tk * a.k + j];
        if (a.wire_ids && lane == 0) reinterpret_cast<int32_t *>(z)[a.k] = a.shift.ids[t];
      } else {
        T *z = static_cast<T *>(a.zout) + t * a.ldzout;
        for (int j = lane; j < a.k; j += 32) z[j] = from_f32<T>(zs[tk * a.k + j]);
      }
    }
  } else {
#pragma unroll
    for (int tk = 0; tk < kGenericTokens; ++tk) {
      const int64_t t = valid[tk] ? t0 + tk : 0;
      if (a.wire) {
        const float *z = static_cast<const float *>(a.zin) + t * a.ldzin;
        for (int j = lane; j < a.k; j += 32) zs[tk * a.k + j] = z[j];
      } else {
        const T *z = static_cast<const T *>(a.zin) + t * a.ldzin;
        for (int j = lane; j < a.k; j += 32) zs[tk * a.k + j] = to_f32(z[j]);
      }
    }
    __syncwarp();
  }

  if (a.dst != nullptr) {
    const T *Ux = a.U2 != nullptr ? static_cast<const T *>(a.U2) : U;
    const int64_t ldux = a.U2 != nullptr ? a.ldu2 : a.ldu;
    const int dx = a.U2 != nullptr ? a.d2 : a.d;
    float ss[kGenericTokens];
#pragma unroll
    for (int tk = 0; tk < kGenericTokens; ++tk) ss[tk] = 0.f;
    for (int i0 = 0; i0 < dx; i0 += kGenericRows) {
      float acc[kGenericTokens][kGenericRows / 32];
#pragma unroll
      for (int tk = 0; tk < kGenericTokens; ++tk)
#pragma unroll
        for (int h = 0; h < kGenericRows / 32; ++h) acc[tk][h] = 0.f;
      for (int j0 = 0; j0 < a.k; j0 += kGenericCoords) {
        stage_u(Ux, ldux, dx, i0, j0);
        const int jn = min(kGenericCoords, a.k - j0);
        for (int jj = 0; jj < jn; ++jj) {
#pragma unroll
          for (int h = 0; h < kGenericRows / 32; ++h) {
            const float u = us[(lane + 32 * h) * kPitch + jj];
#pragma unroll
            for (int tk = 0; tk < kGenericTokens; ++tk) acc[tk][h] = fmaf(zs[tk * a.k + j0 + jj], u, acc[tk][h]);
          }
        }
      }
#pragma unroll
      for (int tk = 0; tk < kGenericTokens; ++tk) {
        if (!valid[tk]) continue;
        T *out = static_cast<T *>(a.dst) + (t0 + tk) * a.lddst;
#pragma unroll
        for (int h = 0; h < kGenericRows / 32; ++h) {
          const int i = i0 + lane + 32 * h;
          if (i >= dx) continue;
          float v = acc[tk][h];
          if (a.add_shift) {
            if (erow[tk]) v += to_f32(erow[tk][i]);
            if (prow[tk]) v += to_f32(prow[tk][i]);
          }
          ss[tk] = fmaf(v, v, ss[tk]);
          out[i] = from_f32<T>(v);
        }
      }
    }
    if (a.rowsumsq != nullptr) {
#pragma unroll
      for (int tk = 0; tk < kGenericTokens; ++tk) {
        float v = ss[tk];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
        if (lane == 0 && valid[tk]) a.rowsumsq[t0 + tk] = v;
      }
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
