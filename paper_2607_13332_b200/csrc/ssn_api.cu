// C-ABI of libssn: argument validation and kernel dispatch.  See include/ssn.h for the
// contract of every entry point.
#include "ssn.h"

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <atomic>
#include <vector>

#include "codec_mma_launch.h"
#include "generic_kernels.cuh"
#include "ssn_common.cuh"

namespace ssn {
namespace {

inline bool valid_dtype(int32_t dt) { return dt == SSN_F32 || dt == SSN_BF16; }

ssn_status_t check_codec(const ssn_codec_t *c) {
  if (c == nullptr || c->U == nullptr) return SSN_ERR_NULL;
  if (!valid_dtype(c->dtype)) return SSN_ERR_DTYPE;
  if (c->d < 1 || c->k < 1 || c->k > c->d || c->ldu < c->k) return SSN_ERR_SHAPE;
  return SSN_OK;
}

// Checks the shared tables when a call uses them and fills the device-side view.
ssn_status_t make_shift(const ssn_codec_t *c, const int32_t *ids, const int32_t *pos,
                        int32_t seq_len, int32_t *dev_status, ShiftTables *out) {
  ShiftTables s{};
  s.E = c->E;
  s.P = c->P;
  s.ids = ids;
  s.pos = pos;
  s.lde = c->lde;
  s.ldp = c->ldp;
  s.vocab = c->vocab;
  s.max_pos = c->max_pos;
  s.seq_len = seq_len;
  s.dev_status = dev_status != nullptr ? dev_status : c->dev_status;
  if (c->E != nullptr) {
    if (ids == nullptr) return SSN_ERR_NULL;
    if (c->lde < c->d || c->vocab < 1) return SSN_ERR_SHAPE;
  }
  if (c->P != nullptr) {
    if (c->ldp < c->d || c->max_pos < 1) return SSN_ERR_SHAPE;
    if (pos == nullptr && seq_len < 1) return SSN_ERR_SHAPE;
  }
  *out = s;
  return SSN_OK;
}

std::atomic<int64_t> g_launches{0};
thread_local int32_t g_last_kernel = SSN_KERNEL_NONE;

// Called after every group of `launches` kernel launches.
ssn_status_t launch_status(int launches = 1) {
  g_launches.fetch_add(launches, std::memory_order_relaxed);
  return cudaGetLastError() == cudaSuccess ? SSN_OK : SSN_ERR_CUDA;
}

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

int sm_count_of_current_device() {
  static int cached[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) n = 0;
    cached[dev] = n;
  }
  return cached[dev];
}

// True when the call can run on the tensor-core kernels: bf16, supported shape, every big
// matrix 16-byte aligned with a leading dimension that keeps its rows 16-byte aligned.
bool mma_eligible(const TokenArgs &a, int32_t dtype) {
  if (dtype != SSN_BF16 || !codec_mma_supports(a.d, a.k)) return false;
  if (!aligned16(a.U) || (a.ldu & 7)) return false;
  if (a.src && (!aligned16(a.src) || (a.lds & 7))) return false;
  if (a.src2 && (!aligned16(a.src2) || (a.lds2 & 7))) return false;
  if (a.dst && (!aligned16(a.dst) || (a.lddst & 7))) return false;
  if (a.sub_shift || a.add_shift) {
    if (a.shift.E && (!aligned16(a.shift.E) || (a.shift.lde & 7))) return false;
    if (a.shift.P && (!aligned16(a.shift.P) || (a.shift.ldp & 7))) return false;
  }
  return true;
}

ssn_status_t launch_generic_token_kernel(const TokenArgs &a, int32_t dtype, cudaStream_t stream) {
  if (a.n == 0) return SSN_OK;
  const int64_t blocks = (a.n + kGenericTokensPerBlock - 1) / kGenericTokensPerBlock;
  if (blocks > 0x7fffffffLL) return SSN_ERR_SHAPE;
  const size_t smem = generic_token_smem_bytes(a.k);
  if (smem > 227 * 1024) return SSN_ERR_SHAPE;   // rank too large for the general kernel's shared memory
  if (smem > 48 * 1024) {
    static std::atomic<uint64_t> configured_f32{0}, configured_bf16{0};
    const cudaError_t e = dtype == SSN_F32 ? allow_dynamic_smem(token_kernel<float>, 227 * 1024, configured_f32)
                                           : allow_dynamic_smem(token_kernel<__nv_bfloat16>, 227 * 1024, configured_bf16);
    if (e != cudaSuccess) {
      cudaGetLastError();
      return SSN_ERR_CUDA;
    }
  }
  if (dtype == SSN_F32)
    token_kernel<float><<<(unsigned)blocks, kGenericWarps * 32, smem, stream>>>(a);
  else
    token_kernel<__nv_bfloat16><<<(unsigned)blocks, kGenericWarps * 32, smem, stream>>>(a);
  g_last_kernel = SSN_KERNEL_GENERIC |
                  ((((a.sub_shift || a.add_shift) && a.shift.E ? SSN_KVAR_E : 0) |
                    ((a.sub_shift || a.add_shift) && a.shift.P ? SSN_KVAR_P : 0) |
                    (a.rowsumsq != nullptr ? SSN_KVAR_ROWSUMSQ : 0)) << 8);
  return launch_status();
}

ssn_status_t launch_token_kernel(const TokenArgs &a, int32_t dtype, cudaStream_t stream) {
  if (a.n == 0) return SSN_OK;
  // wire rows: the tensor-core path takes the projection only (and falls back when it refuses)
  const bool wire_ok = !(a.wire || a.src2) || (a.src != nullptr && a.dst == nullptr);
  // the row statistic: only the plain expansion (no wire rows) on the tensor cores
  const bool stat_ok = a.rowsumsq == nullptr || (a.src == nullptr && a.dst != nullptr && !a.wire);
  if (wire_ok && stat_ok && mma_eligible(a, dtype)) {
    const int sms = sm_count_of_current_device();
    if (sms > 0) {
      MmaArgs m{};
      m.src = static_cast<const __nv_bfloat16 *>(a.src);
      m.zin = static_cast<const __nv_bfloat16 *>(a.zin);
      if (a.wire) {
        m.zout32 = static_cast<float *>(a.zout);
        m.ldzout32 = a.ldzout;
        m.wire_ids = a.wire_ids ? a.shift.ids : nullptr;
      } else {
        m.zout = static_cast<__nv_bfloat16 *>(a.zout);
      }
      m.dst = static_cast<__nv_bfloat16 *>(a.dst);
      m.U = static_cast<const __nv_bfloat16 *>(a.U);
      m.src2 = static_cast<const __nv_bfloat16 *>(a.src2);
      m.lds2 = a.lds2;
      m.rowsumsq = a.rowsumsq;
      m.lds = a.lds;
      m.ldzin = a.ldzin;
      m.ldzout = a.ldzout;
      m.lddst = a.lddst;
      m.ldu = a.ldu;
      m.n = a.n;
      m.d = a.d;
      m.k = a.k;
      m.shift = a.shift;
      const bool shift = (a.sub_shift || a.add_shift) && (a.shift.E || a.shift.P);
      const int mode = (a.src ? 1 : 0) | (a.dst ? 2 : 0);
      cudaError_t e = launch_codec_mma(m, shift, mode, sms, stream);
      if (!((a.wire || a.src2 || a.rowsumsq) && e == cudaErrorNotSupported)) {
        g_launches.fetch_add(1, std::memory_order_relaxed);
        return e == cudaSuccess ? SSN_OK : SSN_ERR_CUDA;
      }
    }
  }
  return launch_generic_token_kernel(a, dtype, stream);
}

}  // namespace

void note_kernel(int family, int variant) { g_last_kernel = family | (variant << 8); }
void count_launches(int launches) { g_launches.fetch_add(launches, std::memory_order_relaxed); }

}  // namespace ssn

namespace ssn {
namespace {
// RIGHT re-projection of `count` matrices [rows[i] x d]: groups of up to kMaxFusedMatrices go to the fused
// tcgen05 kernel in one launch each; what that kernel does not take goes matrix by matrix.
ssn_status_t reproject_right_list(const ssn_codec_t *codec, void *const *W_ptrs, const int64_t *rows,
                                  const int64_t *ldw, int32_t count, cudaStream_t s) {
  const int sms = sm_count_of_current_device();
  int32_t done = 0;
  while (done < count) {
    const int32_t take = count - done < kMaxFusedMatrices ? count - done : kMaxFusedMatrices;
    bool fused = false;
    if (codec->dtype == SSN_BF16 && sms > 0 && aligned16(codec->U) && (codec->ldu & 7) == 0) {
      MmaArgs m{};
      m.U = static_cast<const __nv_bfloat16 *>(codec->U);
      m.ldu = codec->ldu;
      m.d = codec->d;
      m.k = codec->k;
      m.shift.dev_status = codec->dev_status;
      const __nv_bfloat16 *src[kMaxFusedMatrices];
      __nv_bfloat16 *dst[kMaxFusedMatrices];
      for (int32_t i = 0; i < take; ++i) src[i] = dst[i] = static_cast<__nv_bfloat16 *>(W_ptrs[done + i]);
      cudaError_t e = launch_codec_umma_roundtrip_list(m, src, dst, rows + done, ldw + done, ldw + done, take,
                                                       sms, s, false);
      if (e == cudaSuccess) {
        g_launches.fetch_add(1, std::memory_order_relaxed);
        fused = true;
      } else if (e != cudaErrorNotSupported) {
        return SSN_ERR_CUDA;
      }
    }
    if (!fused) {
      // Every row of W is one "token": project onto U and expand again, no shift terms.
      for (int32_t b = done; b < done + take; ++b) {
        TokenArgs a{};
        a.src = W_ptrs[b];
        a.lds = ldw[b];
        a.dst = W_ptrs[b];
        a.lddst = ldw[b];
        a.U = codec->U;
        a.ldu = codec->ldu;
        a.n = rows[b];
        a.d = codec->d;
        a.k = codec->k;
        a.shift.dev_status = codec->dev_status;
        ssn_status_t st = launch_token_kernel(a, codec->dtype, s);
        if (st != SSN_OK) return st;
      }
    }
    done += take;
  }
  return SSN_OK;
}
}  // namespace
}  // namespace ssn

namespace ssn {
namespace {
// LEFT re-projection of up to kMaxFusedMatrices weights [d x cols[i]] on the fused tcgen05 kernel; false when
// that kernel does not take the call (nothing launched).
bool try_reproject_left_fused(const ssn_codec_t *codec, void *const *W_ptrs, const int64_t *cols,
                              const int64_t *ldw, int32_t count, cudaStream_t s, ssn_status_t *st) {
  *st = SSN_OK;
  const int sms = sm_count_of_current_device();
  if (codec->dtype != SSN_BF16 || sms <= 0 || !aligned16(codec->U) || (codec->ldu & 7) != 0) return false;
  MmaArgs m{};
  m.U = static_cast<const __nv_bfloat16 *>(codec->U);
  m.ldu = codec->ldu;
  m.d = codec->d;
  m.k = codec->k;
  m.shift.dev_status = codec->dev_status;
  const __nv_bfloat16 *src[kMaxFusedMatrices];
  __nv_bfloat16 *dst[kMaxFusedMatrices];
  for (int32_t i = 0; i < count; ++i) src[i] = dst[i] = static_cast<__nv_bfloat16 *>(W_ptrs[i]);
  cudaError_t e = launch_codec_umma_roundtrip_list(m, src, dst, cols, ldw, ldw, count, sms, s, true);
  if (e == cudaErrorNotSupported) return false;
  if (e == cudaSuccess)
    g_launches.fetch_add(1, std::memory_order_relaxed);
  else
    *st = SSN_ERR_CUDA;
  return true;
}

// LEFT re-projection of one weight with the general two-kernel form (T = U^T W in the workspace).
ssn_status_t reproject_left_general(const ssn_codec_t *codec, void *W, int64_t cols, int64_t ldw,
                                    void *workspace, size_t workspace_bytes, cudaStream_t s) {
  if (workspace == nullptr || workspace_bytes < (size_t)codec->k * (size_t)cols * sizeof(float))
    return SSN_ERR_WORKSPACE;
  const int64_t col_blocks = (cols + kLeftCols - 1) / kLeftCols;
  if (col_blocks > 0x7fffffffLL || ((int64_t)codec->d + 31) / 32 > 65535) return SSN_ERR_SHAPE;
  LeftArgs a{};
  a.W = W;
  a.U = codec->U;
  a.T = static_cast<float *>(workspace);
  a.ldw = ldw;
  a.ldu = codec->ldu;
  a.m = cols;
  a.d = codec->d;
  a.k = codec->k;
  dim3 g1((unsigned)col_blocks, (unsigned)((codec->k + kGenericKChunk - 1) / kGenericKChunk));
  dim3 g2((unsigned)col_blocks, (unsigned)((codec->d + 31) / 32));
  if (codec->dtype == SSN_F32) {
    left_reduce_kernel<float><<<g1, kLeftCols, 0, s>>>(a);
    left_expand_kernel<float><<<g2, kLeftCols, 0, s>>>(a);
  } else {
    left_reduce_kernel<__nv_bfloat16><<<g1, kLeftCols, 0, s>>>(a);
    left_expand_kernel<__nv_bfloat16><<<g2, kLeftCols, 0, s>>>(a);
  }
  g_last_kernel = SSN_KERNEL_GENERIC;
  return launch_status(2);
}

// LEFT re-projection of `count` weights [d x cols[i]]: groups of up to kMaxFusedMatrices on the fused kernel, the
// rest one by one through the workspace.
ssn_status_t reproject_left_list(const ssn_codec_t *codec, void *const *W_ptrs, const int64_t *cols,
                                 const int64_t *ldw, int32_t count, void *workspace,
                                 size_t workspace_bytes, cudaStream_t s) {
  int32_t done = 0;
  while (done < count) {
    const int32_t take = count - done < kMaxFusedMatrices ? count - done : kMaxFusedMatrices;
    ssn_status_t st;
    if (try_reproject_left_fused(codec, W_ptrs + done, cols + done, ldw + done, take, s, &st)) {
      if (st != SSN_OK) return st;
    } else {
      for (int32_t b = done; b < done + take; ++b) {
        st = reproject_left_general(codec, W_ptrs[b], cols[b], ldw[b], workspace, workspace_bytes, s);
        if (st != SSN_OK) return st;
      }
    }
    done += take;
  }
  return SSN_OK;
}
}  // namespace
}  // namespace ssn

using namespace ssn;

extern "C" {

ssn_status_t ssn_compress(const ssn_codec_t *codec, const void *X, int64_t ldx,
                          const int32_t *ids, const int32_t *pos, int64_t n_tokens,
                          int32_t seq_len, void *Z, int64_t ldz, int32_t *dev_status,
                          void *stream) {
  ssn_status_t st = check_codec(codec);
  if (st != SSN_OK) return st;
  if (n_tokens < 0 || ldx < codec->d || ldz < codec->k) return SSN_ERR_SHAPE;
  if (n_tokens == 0) return SSN_OK;
  if (X == nullptr || Z == nullptr) return SSN_ERR_NULL;
  TokenArgs a{};
  st = make_shift(codec, ids, pos, seq_len, dev_status, &a.shift);
  if (st != SSN_OK) return st;
  a.src = X;
  a.lds = ldx;
  a.zout = Z;
  a.ldzout = ldz;
  a.U = codec->U;
  a.ldu = codec->ldu;
  a.n = n_tokens;
  a.d = codec->d;
  a.k = codec->k;
  a.sub_shift = 1;
  // prepared tables: only kernels that know them read them, the others use E and P
  if (codec->E != nullptr && codec->EU != nullptr) {
    if (codec->ldeu < codec->k) return SSN_ERR_SHAPE;
    a.shift.EU = codec->EU;
    a.shift.ldeu = codec->ldeu;
  }
  if (codec->P != nullptr && codec->PU != nullptr) {
    if (codec->ldpu < codec->k) return SSN_ERR_SHAPE;
    a.shift.PU = codec->PU;
    a.shift.ldpu = codec->ldpu;
  }
  return launch_token_kernel(a, codec->dtype, static_cast<cudaStream_t>(stream));
}

ssn_status_t ssn_prepare_tables(const ssn_codec_t *codec, float *EU, int64_t ldeu, float *PU,
                                int64_t ldpu, void *stream) {
  ssn_status_t st = check_codec(codec);
  if (st != SSN_OK) return st;
  if ((EU != nullptr && codec->E == nullptr) || (PU != nullptr && codec->P == nullptr)) return SSN_ERR_NULL;
  if ((EU != nullptr && (ldeu < codec->k || codec->lde < codec->d || codec->vocab < 1)) ||
      (PU != nullptr && (ldpu < codec->k || codec->ldp < codec->d || codec->max_pos < 1)))
    return SSN_ERR_SHAPE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  for (int which = 0; which < 2; ++which) {
    float *out = which == 0 ? EU : PU;
    if (out == nullptr) continue;
    TableArgs t{};
    t.rows_in = which == 0 ? codec->E : codec->P;
    t.ld_in = which == 0 ? codec->lde : codec->ldp;
    t.n = which == 0 ? codec->vocab : (int64_t)codec->max_pos;
    t.U = codec->U;
    t.ldu = codec->ldu;
    t.out = out;
    t.ld_out = which == 0 ? ldeu : ldpu;
    t.d = codec->d;
    t.k = codec->k;
    const int64_t blocks = (t.n + kTableWarps - 1) / kTableWarps;
    if (blocks > 0x7fffffffLL) return SSN_ERR_SHAPE;
    if (codec->dtype == SSN_F32)
      table_project_kernel<float><<<(unsigned)blocks, kTableWarps * 32, 0, s>>>(t);
    else
      table_project_kernel<__nv_bfloat16><<<(unsigned)blocks, kTableWarps * 32, 0, s>>>(t);
    st = launch_status();
    if (st != SSN_OK) return st;
  }
  return SSN_OK;
}

ssn_status_t ssn_decompress(const ssn_codec_t *codec, const void *Z, int64_t ldz,
                            const int32_t *ids, const int32_t *pos, int64_t n_tokens,
                            int32_t seq_len, void *Xhat, int64_t ldx, int32_t *dev_status,
                            void *stream) {
  ssn_status_t st = check_codec(codec);
  if (st != SSN_OK) return st;
  if (n_tokens < 0 || ldx < codec->d || ldz < codec->k) return SSN_ERR_SHAPE;
  if (n_tokens == 0) return SSN_OK;
  if (Xhat == nullptr || Z == nullptr) return SSN_ERR_NULL;
  TokenArgs a{};
  st = make_shift(codec, ids, pos, seq_len, dev_status, &a.shift);
  if (st != SSN_OK) return st;
  a.zin = Z;
  a.ldzin = ldz;
  a.dst = Xhat;
  a.lddst = ldx;
  a.U = codec->U;
  a.ldu = codec->ldu;
  a.n = n_tokens;
  a.d = codec->d;
  a.k = codec->k;
  a.add_shift = 1;
  return launch_token_kernel(a, codec->dtype, static_cast<cudaStream_t>(stream));
}

ssn_status_t ssn_decompress_rowsumsq(const ssn_codec_t *codec, const void *Z, int64_t ldz,
                                     const int32_t *ids, const int32_t *pos, int64_t n_tokens,
                                     int32_t seq_len, void *Xhat, int64_t ldx, float *rowsumsq,
                                     int32_t *dev_status, void *stream) {
  ssn_status_t st = check_codec(codec);
  if (st != SSN_OK) return st;
  if (n_tokens < 0 || ldx < codec->d || ldz < codec->k) return SSN_ERR_SHAPE;
  if (n_tokens == 0) return SSN_OK;
  if (Xhat == nullptr || Z == nullptr || rowsumsq == nullptr) return SSN_ERR_NULL;
  TokenArgs a{};
  st = make_shift(codec, ids, pos, seq_len, dev_status, &a.shift);
  if (st != SSN_OK) return st;
  a.zin = Z;
  a.ldzin = ldz;
  a.dst = Xhat;
  a.lddst = ldx;
  a.U = codec->U;
  a.ldu = codec->ldu;
  a.n = n_tokens;
  a.d = codec->d;
  a.k = codec->k;
  a.add_shift = 1;
  a.rowsumsq = rowsumsq;
  // the tensor-core kernel adds per-chunk partial sums atomically: start from zero
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(rowsumsq, 0, (size_t)n_tokens * sizeof(float), s) != cudaSuccess) {
    cudaGetLastError();
    return SSN_ERR_CUDA;
  }
  return launch_token_kernel(a, codec->dtype, s);
}

ssn_status_t ssn_grad_project(const ssn_codec_t *codec, const void *G, int64_t ldg,
                              int64_t n_tokens, int32_t mode, void *dZ, int64_t ldz,
                              void *Gpar, int64_t ldgp, void *stream) {
  ssn_status_t st = check_codec(codec);
  if (st != SSN_OK) return st;
  if ((mode & ~(SSN_GRAD_COEFF | SSN_GRAD_FULL)) != 0 || mode == 0) return SSN_ERR_DTYPE;
  if (n_tokens < 0 || ldg < codec->d) return SSN_ERR_SHAPE;
  if ((mode & SSN_GRAD_COEFF) && ldz < codec->k) return SSN_ERR_SHAPE;
  if ((mode & SSN_GRAD_FULL) && ldgp < codec->d) return SSN_ERR_SHAPE;
  if (n_tokens == 0) return SSN_OK;
  if (G == nullptr) return SSN_ERR_NULL;
  if ((mode & SSN_GRAD_COEFF) && dZ == nullptr) return SSN_ERR_NULL;
  if ((mode & SSN_GRAD_FULL) && Gpar == nullptr) return SSN_ERR_NULL;
  TokenArgs a{};
  a.src = G;
  a.lds = ldg;
  if (mode & SSN_GRAD_COEFF) {
    a.zout = dZ;
    a.ldzout = ldz;
  }
  if (mode & SSN_GRAD_FULL) {
    a.dst = Gpar;
    a.lddst = ldgp;
  }
  a.U = codec->U;
  a.ldu = codec->ldu;
  a.n = n_tokens;
  a.d = codec->d;
  a.k = codec->k;
  a.shift.dev_status = codec->dev_status;
  return launch_token_kernel(a, codec->dtype, static_cast<cudaStream_t>(stream));
}

// ---- wire rows ------------------------------------------------------------------------------
namespace {
inline size_t round256(size_t b) { return (b + 255) & ~(size_t)255; }
inline int32_t padded_rank(int32_t k) { return (k + 7) & ~7; }
// the tensor-core kernels take the fp32 coordinates as (head | remainder) of rank 2 * padded k
inline bool wire_split_fits(const ssn_codec_t *c) { return c->dtype == SSN_BF16 && 2 * padded_rank(c->k) <= 128; }
}  // namespace

ssn_status_t ssn_compress_wire(const ssn_codec_t *codec, const void *X, int64_t ldx,
                               const int32_t *ids, const int32_t *pos, int64_t n_tokens,
                               int32_t seq_len, void *wire, int64_t ldw, int32_t with_ids,
                               int32_t *dev_status, void *stream) {
  ssn_status_t st = check_codec(codec);
  if (st != SSN_OK) return st;
  if (n_tokens < 0 || ldx < codec->d || ldw < (int64_t)codec->k + (with_ids ? 1 : 0)) return SSN_ERR_SHAPE;
  if (with_ids && ids == nullptr) return SSN_ERR_NULL;
  if (n_tokens == 0) return SSN_OK;
  if (X == nullptr || wire == nullptr) return SSN_ERR_NULL;
  TokenArgs a{};
  st = make_shift(codec, ids, pos, seq_len, dev_status, &a.shift);
  if (st != SSN_OK) return st;
  a.src = X;
  a.lds = ldx;
  a.zout = wire;
  a.ldzout = ldw;
  a.wire = 1;
  a.wire_ids = with_ids ? 1 : 0;
  a.U = codec->U;
  a.ldu = codec->ldu;
  a.n = n_tokens;
  a.d = codec->d;
  a.k = codec->k;
  a.sub_shift = 1;
  if (codec->E != nullptr && codec->EU != nullptr) {
    if (codec->ldeu < codec->k) return SSN_ERR_SHAPE;
    a.shift.EU = codec->EU;
    a.shift.ldeu = codec->ldeu;
  }
  if (codec->P != nullptr && codec->PU != nullptr) {
    if (codec->ldpu < codec->k) return SSN_ERR_SHAPE;
    a.shift.PU = codec->PU;
    a.shift.ldpu = codec->ldpu;
  }
  return launch_token_kernel(a, codec->dtype, static_cast<cudaStream_t>(stream));
}

ssn_status_t ssn_compress_sum(const ssn_codec_t *codec, const void *X, int64_t ldx, const void *R,
                              int64_t ldr, const int32_t *ids, const int32_t *pos, int64_t n_tokens,
                              int32_t seq_len, void *out, int64_t ldout, int32_t out_form,
                              int32_t *dev_status, void *stream) {
  ssn_status_t st = check_codec(codec);
  if (st != SSN_OK) return st;
  if (out_form != SSN_OUT_STORAGE && out_form != SSN_OUT_WIRE && out_form != SSN_OUT_WIRE_IDS) return SSN_ERR_DTYPE;
  const bool with_ids = out_form == SSN_OUT_WIRE_IDS;
  if (n_tokens < 0 || ldx < codec->d || ldr < codec->d || ldout < (int64_t)codec->k + (with_ids ? 1 : 0))
    return SSN_ERR_SHAPE;
  if (with_ids && ids == nullptr) return SSN_ERR_NULL;
  if (n_tokens == 0) return SSN_OK;
  if (X == nullptr || R == nullptr || out == nullptr) return SSN_ERR_NULL;
  TokenArgs a{};
  st = make_shift(codec, ids, pos, seq_len, dev_status, &a.shift);
  if (st != SSN_OK) return st;
  a.src = X;
  a.lds = ldx;
  a.src2 = R;
  a.lds2 = ldr;
  a.zout = out;
  a.ldzout = ldout;
  a.wire = out_form != SSN_OUT_STORAGE ? 1 : 0;
  a.wire_ids = with_ids ? 1 : 0;
  a.U = codec->U;
  a.ldu = codec->ldu;
  a.n = n_tokens;
  a.d = codec->d;
  a.k = codec->k;
  a.sub_shift = 1;
  if (codec->E != nullptr && codec->EU != nullptr) {
    if (codec->ldeu < codec->k) return SSN_ERR_SHAPE;
    a.shift.EU = codec->EU;
    a.shift.ldeu = codec->ldeu;
  }
  if (codec->P != nullptr && codec->PU != nullptr) {
    if (codec->ldpu < codec->k) return SSN_ERR_SHAPE;
    a.shift.PU = codec->PU;
    a.shift.ldpu = codec->ldpu;
  }
  return launch_token_kernel(a, codec->dtype, static_cast<cudaStream_t>(stream));
}

ssn_status_t ssn_grad_project_wire(const ssn_codec_t *codec, const void *G, int64_t ldg,
                                   int64_t n_tokens, float *dZ, int64_t ldw, void *stream) {
  ssn_status_t st = check_codec(codec);
  if (st != SSN_OK) return st;
  if (n_tokens < 0 || ldg < codec->d || ldw < codec->k) return SSN_ERR_SHAPE;
  if (n_tokens == 0) return SSN_OK;
  if (G == nullptr || dZ == nullptr) return SSN_ERR_NULL;
  TokenArgs a{};
  a.src = G;
  a.lds = ldg;
  a.zout = dZ;
  a.ldzout = ldw;
  a.wire = 1;
  a.U = codec->U;
  a.ldu = codec->ldu;
  a.n = n_tokens;
  a.d = codec->d;
  a.k = codec->k;
  a.shift.dev_status = codec->dev_status;
  return launch_token_kernel(a, codec->dtype, static_cast<cudaStream_t>(stream));
}

size_t ssn_decompress_wire_workspace_bytes(const ssn_codec_t *codec, int64_t n_tokens, int32_t with_ids) {
  if (check_codec(codec) != SSN_OK || n_tokens < 0) return 0;
  size_t bytes = with_ids ? round256((size_t)n_tokens * sizeof(int32_t)) : 0;
  if (wire_split_fits(codec)) {
    const size_t kp2 = 2 * (size_t)padded_rank(codec->k);
    bytes += round256((size_t)n_tokens * kp2 * 2) + round256((size_t)codec->d * kp2 * 2);
  }
  return bytes;
}

ssn_status_t ssn_decompress_wire(const ssn_codec_t *codec, const void *wire, int64_t ldw,
                                 int32_t with_ids, const int32_t *ids, const int32_t *pos,
                                 int64_t n_tokens, int32_t seq_len, void *Xhat, int64_t ldx,
                                 void *workspace, size_t workspace_bytes, int32_t *dev_status,
                                 void *stream) {
  ssn_status_t st = check_codec(codec);
  if (st != SSN_OK) return st;
  if (n_tokens < 0 || ldx < codec->d || ldw < (int64_t)codec->k + (with_ids ? 1 : 0)) return SSN_ERR_SHAPE;
  if (n_tokens == 0) return SSN_OK;
  if (Xhat == nullptr || wire == nullptr) return SSN_ERR_NULL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t ids_bytes = with_ids ? round256((size_t)n_tokens * sizeof(int32_t)) : 0;
  if (with_ids && (workspace == nullptr || workspace_bytes < ids_bytes)) return SSN_ERR_WORKSPACE;
  unsigned char *ws = static_cast<unsigned char *>(workspace);
  int32_t *ids_out = with_ids ? reinterpret_cast<int32_t *>(ws) : nullptr;
  const int32_t kp = padded_rank(codec->k);
  const size_t split_bytes = round256((size_t)n_tokens * 2 * kp * 2), u2_bytes = round256((size_t)codec->d * 2 * kp * 2);
  const bool split = wire_split_fits(codec) && workspace != nullptr && (reinterpret_cast<uintptr_t>(workspace) & 255) == 0 &&
                     workspace_bytes >= ids_bytes + split_bytes + u2_bytes;
  TokenArgs a{};
  st = make_shift(codec, with_ids ? ids_out : ids, pos, seq_len, dev_status, &a.shift);
  if (st != SSN_OK) return st;
  a.dst = Xhat;
  a.lddst = ldx;
  a.n = n_tokens;
  a.d = codec->d;
  a.add_shift = 1;
  if (split || ids_out != nullptr) {
    // one small launch: the ids out of the rows, and for the split form the two bf16 operands
    WirePrepareArgs w{};
    w.wire = static_cast<const float *>(wire);
    w.ldw = ldw;
    w.n = n_tokens;
    w.k = codec->k;
    w.kp = split ? kp : 1;
    w.d = codec->d;
    w.ids = ids_out;
    const int rows_per_block = 256 / w.kp;
    const int64_t split_blocks = (n_tokens + rows_per_block - 1) / rows_per_block;
    const int64_t basis_blocks = split ? (codec->d + rows_per_block - 1) / rows_per_block : 0;
    if (split_blocks + basis_blocks > 0x7fffffffLL) return SSN_ERR_SHAPE;
    w.split_blocks = (int32_t)split_blocks;
    if (split) {
      w.split = reinterpret_cast<__nv_bfloat16 *>(ws + ids_bytes);
      w.U = static_cast<const __nv_bfloat16 *>(codec->U);
      w.ldu = codec->ldu;
      w.U2 = reinterpret_cast<__nv_bfloat16 *>(ws + ids_bytes + split_bytes);
    }
    wire_prepare_kernel<<<(unsigned)(split_blocks + basis_blocks), dim3((unsigned)w.kp, (unsigned)rows_per_block), 0, s>>>(w);
    st = launch_status();
    if (st != SSN_OK) return st;
    if (split) {
      // First choice: the tcgen05 expansion with the head and the remainder as two runs against
      // the same chunk of U (rank k, the basis as it is).  It refuses what it does not take.
      const int sms = sm_count_of_current_device();
      const auto ok16 = [](const void *p, int64_t ld) { return p == nullptr || (aligned16(p) && (ld & 7) == 0); };
      if (sms > 0 && codec->k <= 64 && ok16(codec->U, codec->ldu) && ok16(Xhat, ldx) && ok16(codec->E, codec->lde) &&
          ok16(codec->P, codec->ldp)) {
        MmaArgs m{};
        m.zin = w.split;
        m.zin2 = w.split + kp;
        m.ldzin = 2 * kp;
        m.dst = static_cast<__nv_bfloat16 *>(Xhat);
        m.lddst = ldx;
        m.U = static_cast<const __nv_bfloat16 *>(codec->U);
        m.ldu = codec->ldu;
        m.n = n_tokens;
        m.d = codec->d;
        m.k = codec->k;
        m.shift = a.shift;
        const cudaError_t e = launch_codec_umma_expand(m, a.shift.E != nullptr || a.shift.P != nullptr, sms, s);
        if (e == cudaSuccess) return launch_status();
        if (e != cudaErrorNotSupported) {
          cudaGetLastError();
          return SSN_ERR_CUDA;
        }
      }
      // otherwise rank 2 kp on whichever kernel takes it: (head | rem)(U | U)^T = (head + rem) U^T
      a.zin = w.split;
      a.ldzin = 2 * kp;
      a.U = w.U2;
      a.ldu = 2 * kp;
      a.k = 2 * kp;
    }
  }
  if (!split) {
    a.zin = wire;
    a.ldzin = ldw;
    a.wire = 1;
    a.U = codec->U;
    a.ldu = codec->ldu;
    a.k = codec->k;
  }
  return launch_token_kernel(a, codec->dtype, s);
}

ssn_status_t ssn_reparam_project(const ssn_codec_t *codec, const void *H, int64_t ldh, int64_t m,
                                 const void *Zw, int64_t ldzw, int64_t n_tokens, void *Y,
                                 int64_t ldy, void *coords, int64_t ldc, void *stream) {
  ssn_status_t st = check_codec(codec);
  if (st != SSN_OK) return st;
  if (n_tokens < 0 || m < 1 || m > 0x7fffffffLL || ldh < m || ldzw < codec->k || ldy < codec->d) return SSN_ERR_SHAPE;
  if (coords != nullptr && ldc < codec->k) return SSN_ERR_SHAPE;
  if (n_tokens == 0) return SSN_OK;
  if (H == nullptr || Zw == nullptr || Y == nullptr) return SSN_ERR_NULL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int sms = sm_count_of_current_device();
  if (codec->dtype == SSN_BF16 && sms > 0 && aligned16(codec->U) && (codec->ldu & 7) == 0 && aligned16(Zw) &&
      (ldzw & 7) == 0 && n_tokens <= 0x7fffffffLL) {
    MmaArgs a{};
    a.U = static_cast<const __nv_bfloat16 *>(codec->U);
    a.ldu = codec->ldu;
    a.d = codec->d;
    a.k = codec->k;
    a.B1 = static_cast<const __nv_bfloat16 *>(Zw);
    a.ldb1 = ldzw;
    a.d1 = (int32_t)m;
    a.zout = static_cast<__nv_bfloat16 *>(coords);
    a.ldzout = ldc;
    a.shift.dev_status = codec->dev_status;
    const __nv_bfloat16 *src = static_cast<const __nv_bfloat16 *>(H);
    __nv_bfloat16 *dst = static_cast<__nv_bfloat16 *>(Y);
    cudaError_t e = launch_codec_umma_roundtrip_list(a, &src, &dst, &n_tokens, &ldh, &ldy, 1, sms, s, false);
    if (e == cudaSuccess) {
      g_launches.fetch_add(1, std::memory_order_relaxed);
      return SSN_OK;
    }
    if (e != cudaErrorNotSupported) return SSN_ERR_CUDA;
  }
  // general path: one launch of the general kernel, the coordinates stay in fp32 in shared memory
  TokenArgs p{};
  p.src = H;
  p.lds = ldh;
  p.zout = coords;
  p.ldzout = ldc;
  p.dst = Y;
  p.lddst = ldy;
  p.U = Zw;           // contraction over the m columns of H
  p.ldu = ldzw;
  p.d = (int32_t)m;
  p.U2 = codec->U;    // expansion to the d columns of Y
  p.ldu2 = codec->ldu;
  p.d2 = codec->d;
  p.n = n_tokens;
  p.k = codec->k;
  return launch_generic_token_kernel(p, codec->dtype, s);
}

ssn_status_t ssn_reparam_grad_factor(const ssn_codec_t *codec, const void *H, int64_t ldh, int64_t m,
                                     const void *dY, int64_t lddy, int64_t n_tokens, float *dZw,
                                     int64_t lddz, void *workspace, size_t workspace_bytes,
                                     void *stream) {
  ssn_status_t st = check_codec(codec);
  if (st != SSN_OK) return st;
  if (n_tokens < 0 || m < 1 || m > 0x7fffffffLL || ldh < m || lddy < codec->d || lddz < codec->k) return SSN_ERR_SHAPE;
  if (dZw == nullptr) return SSN_ERR_NULL;
  if (n_tokens == 0) {   // an empty sum over the tokens
    const cudaError_t e = cudaMemset2DAsync(dZw, (size_t)lddz * sizeof(float), 0, (size_t)codec->k * sizeof(float),
                                            (size_t)m, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? SSN_OK : SSN_ERR_CUDA;
  }
  if (H == nullptr || dY == nullptr) return SSN_ERR_NULL;
  const int32_t kpad = (codec->k + 7) / 8 * 8;
  const size_t esz = codec->dtype == SSN_F32 ? sizeof(float) : sizeof(__nv_bfloat16);
  if (workspace == nullptr || workspace_bytes < (size_t)n_tokens * (size_t)kpad * esz) return SSN_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  TokenArgs p{};      // C = dY U: the same projection as the backward pass of the boundary
  p.src = dY;
  p.lds = lddy;
  p.zout = workspace;
  p.ldzout = kpad;
  p.U = codec->U;
  p.ldu = codec->ldu;
  p.n = n_tokens;
  p.d = codec->d;
  p.k = codec->k;
  p.shift.dev_status = codec->dev_status;
  st = launch_token_kernel(p, codec->dtype, s);
  if (st != SSN_OK) return st;
  const int sms = sm_count_of_current_device();
  if (codec->dtype == SSN_BF16 && sms > 0) {
    cudaError_t e = launch_codec_umma_tokens(static_cast<const __nv_bfloat16 *>(H), ldh,
                                             static_cast<const __nv_bfloat16 *>(workspace), kpad, dZw, lddz,
                                             n_tokens, (int32_t)m, codec->k, codec->dev_status, sms, s);
    if (e == cudaSuccess) {
      g_launches.fetch_add(1, std::memory_order_relaxed);
      return SSN_OK;
    }
    if (e != cudaErrorNotSupported) return SSN_ERR_CUDA;
  }
  TokensContractArgs c{};
  c.H = H;
  c.C = workspace;
  c.out = dZw;
  c.ldh = ldh;
  c.ldc = kpad;
  c.ldout = lddz;
  c.n = n_tokens;
  c.m = (int32_t)m;
  c.k = codec->k;
  dim3 grid((unsigned)((m + 31) / 32), (unsigned)((codec->k + 7) / 8));
  if (codec->dtype == SSN_F32)
    tokens_contract_kernel<float><<<grid, 256, 0, s>>>(c);
  else
    tokens_contract_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>(c);
  return launch_status();
}

ssn_status_t ssn_head_embed(const ssn_codec_t *codec, const void *Elow, int64_t ldel,
                            int64_t vocab_low, const int32_t *ids, const int32_t *pos,
                            int64_t n_tokens, int32_t seq_len, void *X0, int64_t ldx,
                            void *workspace, size_t workspace_bytes, int32_t *dev_status,
                            void *stream) {
  ssn_status_t st = check_codec(codec);
  if (st != SSN_OK) return st;
  if (n_tokens < 0 || vocab_low < 1 || ldel < codec->k || ldx < codec->d) return SSN_ERR_SHAPE;
  if (n_tokens == 0) return SSN_OK;
  if (Elow == nullptr || ids == nullptr || X0 == nullptr) return SSN_ERR_NULL;
  const int32_t kpad = (codec->k + 7) / 8 * 8;
  const size_t esz = codec->dtype == SSN_F32 ? sizeof(float) : sizeof(__nv_bfloat16);
  if (workspace == nullptr || workspace_bytes < (size_t)n_tokens * (size_t)kpad * esz) return SSN_ERR_WORKSPACE;
  GatherArgs g{};
  g.table = Elow;
  g.out = workspace;
  g.ids = ids;
  g.ld_table = ldel;
  g.ld_out = kpad;
  g.n = n_tokens;
  g.rows = vocab_low;
  g.k = codec->k;
  g.kpad = kpad;
  g.dev_status = dev_status != nullptr ? dev_status : codec->dev_status;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (kpad <= 256) {
    const int rows_per_block = 256 / (int)kpad;
    const int64_t blocks = (n_tokens + rows_per_block - 1) / rows_per_block;
    if (blocks > 0x7fffffffLL) return SSN_ERR_SHAPE;
    const dim3 block((unsigned)kpad, (unsigned)rows_per_block);
    if (codec->dtype == SSN_F32)
      gather_rows_2d_kernel<float><<<(unsigned)blocks, block, 0, s>>>(g);
    else
      gather_rows_2d_kernel<__nv_bfloat16><<<(unsigned)blocks, block, 0, s>>>(g);
  } else {
    const int64_t total = n_tokens * kpad, blocks = (total + 255) / 256;
    if (blocks > 0x7fffffffLL) return SSN_ERR_SHAPE;
    if (codec->dtype == SSN_F32)
      gather_rows_kernel<float><<<(unsigned)blocks, 256, 0, s>>>(g);
    else
      gather_rows_kernel<__nv_bfloat16><<<(unsigned)blocks, 256, 0, s>>>(g);
  }
  st = launch_status();
  if (st != SSN_OK) return st;
  return ssn_decompress(codec, workspace, kpad, ids, pos, n_tokens, seq_len, X0, ldx, dev_status, stream);
}

size_t ssn_weight_reproject_workspace_bytes(const ssn_codec_t *codec, int64_t rows,
                                            int64_t cols, int32_t side, int32_t batch) {
  if (check_codec(codec) != SSN_OK || rows < 1 || cols < 1 || batch < 1) return 0;
  if (side == SSN_SIDE_LEFT) return (size_t)codec->k * (size_t)cols * sizeof(float);
  return 0;
}

ssn_status_t ssn_weight_reproject_list(const ssn_codec_t *codec, void *const *W_ptrs,
                                       const int64_t *extent, const int64_t *ldw, int32_t count,
                                       int32_t side, void *workspace, size_t workspace_bytes,
                                       void *stream) {
  ssn_status_t st = check_codec(codec);
  if (st != SSN_OK) return st;
  if (side != SSN_SIDE_LEFT && side != SSN_SIDE_RIGHT) return SSN_ERR_DTYPE;
  if (count < 0) return SSN_ERR_SHAPE;
  if (count == 0) return SSN_OK;
  if (W_ptrs == nullptr || extent == nullptr || ldw == nullptr) return SSN_ERR_NULL;
  for (int32_t b = 0; b < count; ++b) {
    if (W_ptrs[b] == nullptr) return SSN_ERR_NULL;
    if (extent[b] < 1 || ldw[b] < (side == SSN_SIDE_RIGHT ? (int64_t)codec->d : extent[b])) return SSN_ERR_SHAPE;
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (side == SSN_SIDE_RIGHT) return reproject_right_list(codec, W_ptrs, extent, ldw, count, s);
  return reproject_left_list(codec, W_ptrs, extent, ldw, count, workspace, workspace_bytes, s);
}

ssn_status_t ssn_weight_reproject(const ssn_codec_t *codec, void *const *W_ptrs, int32_t batch,
                                  int64_t rows, int64_t cols, int64_t ldw, int32_t side,
                                  void *workspace, size_t workspace_bytes, void *stream) {
  ssn_status_t st = check_codec(codec);
  if (st != SSN_OK) return st;
  if (side != SSN_SIDE_LEFT && side != SSN_SIDE_RIGHT) return SSN_ERR_DTYPE;
  if (batch < 0 || rows < 1 || cols < 1 || ldw < cols) return SSN_ERR_SHAPE;
  if ((side == SSN_SIDE_RIGHT ? cols : rows) != codec->d) return SSN_ERR_SHAPE;
  if (batch == 0) return SSN_OK;
  if (W_ptrs == nullptr) return SSN_ERR_NULL;
  for (int32_t b = 0; b < batch; ++b)
    if (W_ptrs[b] == nullptr) return SSN_ERR_NULL;
  const size_t need = ssn_weight_reproject_workspace_bytes(codec, rows, cols, side, batch);
  if (need > 0 && (workspace == nullptr || workspace_bytes < need)) return SSN_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);

  if (side == SSN_SIDE_RIGHT) {
    std::vector<int64_t> nrows((size_t)batch, rows), lds((size_t)batch, ldw);
    return reproject_right_list(codec, W_ptrs, nrows.data(), lds.data(), batch, s);
  }

  std::vector<int64_t> ncols((size_t)batch, cols), lds((size_t)batch, ldw);
  return reproject_left_list(codec, W_ptrs, ncols.data(), lds.data(), batch, workspace, workspace_bytes, s);
}

const char *ssn_status_string(ssn_status_t status) {
  switch (status) {
    case SSN_OK: return "ok";
    case SSN_ERR_NULL: return "a required pointer is NULL";
    case SSN_ERR_SHAPE: return "impossible size, rank or leading dimension";
    case SSN_ERR_DTYPE: return "unknown element type, side or mode";
    case SSN_ERR_WORKSPACE: return "workspace missing or too small";
    case SSN_ERR_CUDA: return "the CUDA runtime refused a launch";
  }
  return "unknown status";
}

int32_t ssn_version(void) { return SSN_VERSION; }

int64_t ssn_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int32_t ssn_last_kernel(void) { return g_last_kernel; }

ssn_status_t ssn_selftest_bounded_wait(int32_t max_polls, int32_t *dev_status, void *stream) {
  if (dev_status == nullptr) return SSN_ERR_NULL;
  if (max_polls < 1 || max_polls > (1 << 20)) return SSN_ERR_SHAPE;
  const cudaError_t e = launch_bounded_wait_selftest(max_polls, dev_status, static_cast<cudaStream_t>(stream));
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return e == cudaSuccess ? SSN_OK : SSN_ERR_CUDA;
}

}  // extern "C"
