// Instantiations and launcher of the tensor-core codec kernels (see codec_mma.cuh).
#include "codec_mma.cuh"
#include "codec_mma_dsplit.cuh"
#include "codec_expand64.cuh"
#include "codec_umma.cuh"
#include "codec_umma_roundtrip.cuh"
#include "codec_umma_expand.cuh"
#include "codec_umma_tokens.cuh"


#include <cstdlib>
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

template <int NT, int MT, bool SHIFT, int MODE>
cudaError_t launch_dsplit_one(const MmaArgs &a, int sm_count, cudaStream_t stream) {
  auto kernel = codec_mma_dsplit_kernel<NT, MT, SHIFT, MODE>;
  constexpr int smem = DsplitConfig<NT, MT>::kSmemBytes;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  int64_t grid = (a.n + 16 * MT - 1) / (16 * MT);
  if (grid > sm_count) grid = sm_count;
  kernel<<<(unsigned)grid, kMmaThreads, smem, stream>>>(a);
  return cudaGetLastError();
}

template <int NT, int MT>
cudaError_t launch_dsplit_nt(const MmaArgs &a, bool shift, int mode, int sm_count, cudaStream_t s) {
  if (mode == kModeProject)
    return shift ? launch_dsplit_one<NT, MT, true, kModeProject>(a, sm_count, s)
                 : launch_dsplit_one<NT, MT, false, kModeProject>(a, sm_count, s);
  if (mode == kModeExpand)
    return shift ? launch_dsplit_one<NT, MT, true, kModeExpand>(a, sm_count, s)
                 : launch_dsplit_one<NT, MT, false, kModeExpand>(a, sm_count, s);
  return launch_dsplit_one<NT, MT, false, kModeBoth>(a, sm_count, s);
}

template <int MT>
cudaError_t launch_dsplit(const MmaArgs &a, bool shift, int mode, int nt, int sm_count, cudaStream_t s) {
  if (nt <= 1) return launch_dsplit_nt<1, MT>(a, shift, mode, sm_count, s);
  if (nt <= 2) return launch_dsplit_nt<2, MT>(a, shift, mode, sm_count, s);
  if (nt <= 4) return launch_dsplit_nt<4, MT>(a, shift, mode, sm_count, s);
  if (nt <= 5) return launch_dsplit_nt<5, MT>(a, shift, mode, sm_count, s);
  if (nt <= 6) return launch_dsplit_nt<6, MT>(a, shift, mode, sm_count, s);
  return launch_dsplit_nt<8, MT>(a, shift, mode, sm_count, s);
}

template <int NT, int MT, bool SHIFT, bool PDEDUP>
cudaError_t launch_expand64_one(const MmaArgs &a, int sm_count, cudaStream_t stream) {
  auto kernel = codec_expand64_kernel<NT, MT, SHIFT, PDEDUP>;
  constexpr int smem = kStages * UStageRing64<NT>::kStageBytes;
  static bool configured = false;
  if (smem > 48 * 1024 && !configured) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  kernel<<<(unsigned)sm_count, kMmaThreads, smem, stream>>>(a);
  return cudaGetLastError();
}

template <int NT>
cudaError_t launch_expand64_nt(const MmaArgs &a, bool shift, bool dedup, int sm_count, cudaStream_t s) {
  if (!shift) return launch_expand64_one<NT, 2, false, false>(a, sm_count, s);
  if (dedup) return launch_expand64_one<NT, 2, true, true>(a, sm_count, s);
  return launch_expand64_one<NT, 1, true, false>(a, sm_count, s);
}

inline bool aligned32(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 31) == 0; }

// Expansion with 64-column chunks; cudaErrorNotSupported sends the call to the 32-column kernel.
cudaError_t launch_expand64(const MmaArgs &a, bool shift, int sm_count, cudaStream_t stream) {
  const int nt = (a.k + 7) / 8;
  if (a.d % 64 != 0 || nt > 8 || !aligned32(a.dst) || (a.lddst & 15)) return cudaErrorNotSupported;
  bool dedup = false;
  if (shift) {
    if (a.shift.E && (!aligned32(a.shift.E) || (a.shift.lde & 15))) return cudaErrorNotSupported;
    if (a.shift.P && (!aligned32(a.shift.P) || (a.shift.ldp & 15))) return cudaErrorNotSupported;
    // tiles of 16 batch entries at one position: implicit positions, whole sequences, batch % 16 == 0
    dedup = a.shift.P != nullptr && a.shift.pos == nullptr && a.shift.seq_len >= 1 &&
            a.n % a.shift.seq_len == 0 && (a.n / a.shift.seq_len) % 16 == 0;
  }
  if (nt <= 1) return launch_expand64_nt<1>(a, shift, dedup, sm_count, stream);
  if (nt <= 2) return launch_expand64_nt<2>(a, shift, dedup, sm_count, stream);
  if (nt <= 4) return launch_expand64_nt<4>(a, shift, dedup, sm_count, stream);
  if (nt <= 5) return launch_expand64_nt<5>(a, shift, dedup, sm_count, stream);
  if (nt <= 6) return launch_expand64_nt<6>(a, shift, dedup, sm_count, stream);
  return launch_expand64_nt<8>(a, shift, dedup, sm_count, stream);
}

// ---- tcgen05 / TMA projection ---------------------------------------------------------------
using EncodeTiledFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                   const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                   const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
    else
      cudaGetLastError();
  }
  return fn;
}

// Row-major bf16 matrix [rows x cols], leading dimension ld, fetched in boxes of box_rows x 64
// columns into the 128-byte swizzled layout.
bool make_sw128_map(CUtensorMap *map, const void *base, int64_t rows, int64_t cols, int64_t ld,
                    int box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (fn == nullptr || rows < 1 || rows > 0x7fffffffLL) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {(cuuint32_t)kUmmaCols, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box,
            estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Row-major bf16 tensor [n2][n1][cols] (row pitch ld, slab pitch ld2, in elements), fetched in
// boxes of 64 columns x box1 x box2 into the 128-byte swizzled layout.
bool make_sw128_map3(CUtensorMap *map, const void *base, int64_t cols, int64_t n1, int64_t n2, int64_t ld,
                     int64_t ld2, int box1, int box2) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (fn == nullptr || n1 < 1 || n2 < 1 || n1 > 0x7fffffffLL || n2 > 0x7fffffffLL) return false;
  cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)n1, (cuuint64_t)n2};
  cuuint64_t strides[2] = {(cuuint64_t)ld * 2, (cuuint64_t)ld2 * 2};
  cuuint32_t box[3] = {(cuuint32_t)kUmmaCols, (cuuint32_t)box1, (cuuint32_t)box2};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box,
            estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int KG, bool HAS_E, bool HAS_P>
cudaError_t launch_umma_expand_one(const MmaArgs &a, const ExpandGeometry &geo, const UmmaExpandMaps &maps,
                                   int sm_count, cudaStream_t stream) {
  auto kernel = codec_umma_expand_kernel<KG, HAS_E, HAS_P>;
  constexpr int smem = UmmaExpandConfig<KG, HAS_E, HAS_P>::kSmemBytes;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  const int64_t units = geo.ntiles * (a.d / kChunkCols);     // (tile, chunk) pairs, dealt evenly
  int64_t grid = units < sm_count ? units : sm_count;
  kernel<<<(unsigned)grid, kExpandThreads, smem, stream>>>(a, geo, maps);
  return cudaGetLastError();
}

template <int NTP, bool HAS_E, bool HAS_P>
cudaError_t launch_umma_one(const MmaArgs &a, const UmmaMaps &maps, int sm_count, cudaStream_t stream) {
  auto kernel = codec_umma_project_kernel<NTP, HAS_E, HAS_P>;
  constexpr int smem = UmmaProjectConfig<NTP, HAS_E, HAS_P>::kSmemBytes;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  // pairs of CTAs (clusters of two) that share their odd tile; see the kernel's schedule
  const int64_t ntiles = (a.n + kUmmaTile - 1) / kUmmaTile;
  int64_t pairs = ntiles;   // with few tiles every pair has one and splits it over d
  if (pairs > sm_count / 2) pairs = sm_count / 2;
  if (pairs < 1) {   // a single SM: plain launch
    kernel<<<(unsigned)(ntiles < sm_count ? ntiles : sm_count), kUmmaThreads, smem, stream>>>(a, maps);
    return cudaGetLastError();
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(2 * pairs));
  cfg.blockDim = dim3(kUmmaThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, a, maps);
  if (e == cudaSuccess) return e;
  // a device that cannot co-schedule the pairs: the same kernel without clusters
  cudaGetLastError();
  const int64_t grid = ntiles < sm_count ? ntiles : sm_count;
  kernel<<<(unsigned)grid, kUmmaThreads, smem, stream>>>(a, maps);
  return cudaGetLastError();
}

template <int NTP>
cudaError_t launch_umma_ntp(const MmaArgs &a, bool has_e, bool has_p, const UmmaMaps &maps, int sm_count,
                            cudaStream_t s) {
  if (has_e && has_p) return launch_umma_one<NTP, true, true>(a, maps, sm_count, s);
  if (has_e) return launch_umma_one<NTP, true, false>(a, maps, sm_count, s);
  if (has_p) return launch_umma_one<NTP, false, true>(a, maps, sm_count, s);
  return launch_umma_one<NTP, false, false>(a, maps, sm_count, s);
}

}  // namespace

// Projection on tcgen05.  Returns cudaErrorNotSupported when the call should take the mma.sync
// kernel instead: small batches, k > 128, d not a multiple of 64, explicit or
// wrapping positions inside a 128-token tile, no tensor map.
cudaError_t launch_codec_umma_project(const MmaArgs &a, bool shift, int sm_count, cudaStream_t stream) {
  if ((a.zout == nullptr) == (a.zout32 == nullptr) || a.dst != nullptr || a.src == nullptr)
    return cudaErrorNotSupported;
  if (a.d % kUmmaCols != 0 || a.k > 128 || a.n < 4 * kUmmaTile || a.n > 0x7fffffffLL)
    return cudaErrorNotSupported;
  // a term with a prepared table is subtracted in the epilogue and needs no operand
  const bool has_e = shift && a.shift.E != nullptr && a.shift.EU == nullptr;
  const bool has_p = shift && a.shift.P != nullptr && a.shift.PU == nullptr;
  if (has_p && (a.shift.pos != nullptr || a.shift.seq_len % kUmmaTile != 0 ||
                a.shift.seq_len > a.shift.max_pos))
    return cudaErrorNotSupported;
  const int ntp = 2 * ((a.k + 15) / 16);
  MmaArgs b = a;
  if (!shift) b.shift.EU = b.shift.PU = nullptr;
  // whole sequences of 128-position blocks: tiles of one block share their positional product
  b.pshare = has_e && has_p && a.k <= 64 && a.n % a.shift.seq_len == 0 ? 1 : 0;
  UmmaMaps maps;
  if (!make_sw128_map(&maps.x, a.src, a.n, a.d, a.lds, kUmmaTile)) return cudaErrorNotSupported;
  if (!make_sw128_map(&maps.u, a.U, a.d, a.k, a.ldu, kUmmaCols)) return cudaErrorNotSupported;
  if (!make_sw128_map(&maps.u_wide, a.U, a.d, a.k <= 64 ? 64 : 128, a.ldu, kUmmaCols))
    return cudaErrorNotSupported;
  maps.p = maps.x;
  maps.x2 = maps.x;
  if (a.src2 != nullptr) {   // a second addend: only the launches without row operands take it
    if (has_e || has_p) return cudaErrorNotSupported;
    if (!make_sw128_map(&maps.x2, a.src2, a.n, a.d, a.lds2, kUmmaTile)) return cudaErrorNotSupported;
  }
  if (has_p && !make_sw128_map(&maps.p, a.shift.P, a.shift.max_pos, a.d, a.shift.ldp, kUmmaTile))
    return cudaErrorNotSupported;
  if (ntp <= 2) return launch_umma_ntp<2>(b, has_e, has_p, maps, sm_count, stream);
  if (ntp <= 4) return launch_umma_ntp<4>(b, has_e, has_p, maps, sm_count, stream);
  if (ntp <= 6) return launch_umma_ntp<6>(b, has_e, has_p, maps, sm_count, stream);
  if (ntp <= 8) return launch_umma_ntp<8>(b, has_e, has_p, maps, sm_count, stream);
  if (ntp <= 12) return launch_umma_ntp<12>(b, has_e, has_p, maps, sm_count, stream);
  return launch_umma_ntp<16>(b, has_e, has_p, maps, sm_count, stream);
}

namespace {
template <int NTP, bool LEFT>
cudaError_t launch_roundtrip_ntp(const MmaArgs &a, const UmmaRoundTripMaps &maps, int sm_count, cudaStream_t stream) {
  auto kernel = codec_umma_roundtrip_kernel<NTP, LEFT>;
  constexpr int smem = UmmaRoundTripConfig<NTP>::kSmemBytes;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  int64_t grid = maps.tile_start[maps.count];
  if (grid > sm_count) grid = sm_count;
  kernel<<<(unsigned)grid, kRoundTripThreads, smem, stream>>>(a, maps);
  return cudaGetLastError();
}
}  // namespace

// Project-then-expand on tcgen05 for `count` matrices [rows[i] x d] at once (src[i] -> dst[i], which
// may be the same buffer).  Returns cudaErrorNotSupported when the call should take the mma.sync
// kernels instead: k > 128, d not a multiple of 128, few rows in all, too many matrices, no tensor map
// (unaligned base or leading dimension).  zout (coordinates, bf16) only with one matrix.
cudaError_t launch_codec_umma_roundtrip_list(const MmaArgs &a, const __nv_bfloat16 *const *src,
                                             __nv_bfloat16 *const *dst, const int64_t *rows,
                                             const int64_t *lds, const int64_t *lddst, int count,
                                             int sm_count, cudaStream_t stream, bool left) {
  if (count < 1 || count > kRoundTripMaxMatrices) return cudaErrorNotSupported;
  if (a.d % kChunkCols != 0 || a.k > 128) return cudaErrorNotSupported;
  UmmaRoundTripMaps maps;
  int64_t tiles = 0, total = 0;
  for (int i = 0; i < count; ++i) {
    if (src[i] == nullptr || dst[i] == nullptr || rows[i] < 1 || rows[i] > 0x7fffffffLL) return cudaErrorNotSupported;
    maps.tile_start[i] = (int32_t)tiles;
    maps.rows[i] = rows[i];
    tiles += (rows[i] + kUmmaTile - 1) / kUmmaTile;
    total += rows[i];
    if (tiles > 0x3fffffffLL) return cudaErrorNotSupported;
    if (left) {   // [d x rows[i]]: `rows` counts the columns, which are what a tile spans
      if (!make_sw128_map(&maps.s[i], src[i], a.d, rows[i], lds[i], kUmmaCols)) return cudaErrorNotSupported;
      if (!make_sw128_map(&maps.out[i], dst[i], a.d, rows[i], lddst[i], 32)) return cudaErrorNotSupported;
    } else {
      if (!make_sw128_map(&maps.s[i], src[i], rows[i], a.B1 != nullptr ? a.d1 : a.d, lds[i], kUmmaTile))
        return cudaErrorNotSupported;
      if (!make_sw128_map(&maps.out[i], dst[i], rows[i], a.d, lddst[i], 32)) return cudaErrorNotSupported;
    }
  }
  if (total < 4 * kUmmaTile) return cudaErrorNotSupported;
  for (int i = count; i < kRoundTripMaxMatrices; ++i) {
    maps.s[i] = maps.s[0];
    maps.out[i] = maps.out[0];
    maps.rows[i] = 0;
    maps.tile_start[i + 1] = (int32_t)tiles;
  }
  maps.tile_start[count] = (int32_t)tiles;
  maps.count = count;
  if (!make_sw128_map(&maps.u, a.U, a.d, a.k, a.ldu, kUmmaCols)) return cudaErrorNotSupported;
  if (!make_sw128_map(&maps.u_wide, a.U, a.d, a.k <= 64 ? 64 : 128, a.ldu, kUmmaCols)) return cudaErrorNotSupported;
  maps.b1 = maps.u;
  maps.b1_wide = maps.u_wide;
  if (a.B1 != nullptr) {
    if (left || a.d1 < kUmmaCols || a.d1 % kUmmaCols != 0) return cudaErrorNotSupported;
    if (!make_sw128_map(&maps.b1, a.B1, a.d1, a.k, a.ldb1, kUmmaCols)) return cudaErrorNotSupported;
    if (!make_sw128_map(&maps.b1_wide, a.B1, a.d1, a.k <= 64 ? 64 : 128, a.ldb1, kUmmaCols)) return cudaErrorNotSupported;
  }
  MmaArgs b = a;
  if (count > 1 || left) b.zout = nullptr;
  const int ntp = 2 * ((a.k + 15) / 16);
  if (left) {
    if (ntp <= 2) return launch_roundtrip_ntp<2, true>(b, maps, sm_count, stream);
    if (ntp <= 4) return launch_roundtrip_ntp<4, true>(b, maps, sm_count, stream);
    if (ntp <= 6) return launch_roundtrip_ntp<6, true>(b, maps, sm_count, stream);
    if (ntp <= 8) return launch_roundtrip_ntp<8, true>(b, maps, sm_count, stream);
    if (ntp <= 12) return launch_roundtrip_ntp<12, true>(b, maps, sm_count, stream);
    return launch_roundtrip_ntp<16, true>(b, maps, sm_count, stream);
  }
  if (ntp <= 2) return launch_roundtrip_ntp<2, false>(b, maps, sm_count, stream);
  if (ntp <= 4) return launch_roundtrip_ntp<4, false>(b, maps, sm_count, stream);
  if (ntp <= 6) return launch_roundtrip_ntp<6, false>(b, maps, sm_count, stream);
  if (ntp <= 8) return launch_roundtrip_ntp<8, false>(b, maps, sm_count, stream);
  if (ntp <= 12) return launch_roundtrip_ntp<12, false>(b, maps, sm_count, stream);
  return launch_roundtrip_ntp<16, false>(b, maps, sm_count, stream);
}

cudaError_t launch_codec_umma_roundtrip(const MmaArgs &a, int sm_count, cudaStream_t stream) {
  if (a.src == nullptr || a.dst == nullptr || a.n > 0x7fffffffLL) return cudaErrorNotSupported;
  const __nv_bfloat16 *src = a.src;
  __nv_bfloat16 *dst = a.dst;
  return launch_codec_umma_roundtrip_list(a, &src, &dst, &a.n, &a.lds, &a.lddst, 1, sm_count, stream, false);
}

// Expansion (decompress) on tcgen05.  Returns cudaErrorNotSupported when the call should take the
// mma.sync kernel instead: k > 128, d not a multiple of 128, few tokens, no tensor map, or a
// position table with explicit positions / a batch that is not made of groups of 8 whole
// sequences whose length is a multiple of 16.
cudaError_t launch_codec_umma_expand(const MmaArgs &a, bool shift, int sm_count, cudaStream_t stream) {
  if (a.zin == nullptr || a.dst == nullptr || a.src != nullptr) return cudaErrorNotSupported;
  if (a.d % kChunkCols != 0 || a.k > 128 || a.n < 4 * kUmmaTile || a.n > 0x7fffffffLL)
    return cudaErrorNotSupported;
  const bool has_e = shift && a.shift.E != nullptr, has_p = shift && a.shift.P != nullptr;
  ExpandGeometry geo{};
  geo.seq_len = a.shift.seq_len;
  if (has_p) {
    const int64_t L = a.shift.seq_len;
    if (a.shift.pos != nullptr || L < kGridPos || L % kGridPos != 0 || L > a.shift.max_pos || a.n % L != 0 ||
        (a.n / L) % kGridSeqs != 0)
      return cudaErrorNotSupported;
    geo.grid_mode = 1;
    geo.nsg = (int32_t)(a.n / L / kGridSeqs);
    geo.ntiles = (int64_t)geo.nsg * (L / kGridPos);
  } else {
    geo.grid_mode = 0;
    geo.nsg = 1;
    geo.ntiles = (a.n + kUmmaTile - 1) / kUmmaTile;
  }
  UmmaExpandMaps maps;
  if (geo.grid_mode) {
    const int64_t L = a.shift.seq_len, B = a.n / L;
    if (!make_sw128_map3(&maps.z, a.zin, a.k, L, B, a.ldzin, L * a.ldzin, kGridPos, kGridSeqs))
      return cudaErrorNotSupported;
    if (!make_sw128_map3(&maps.out, a.dst, a.d, L, B, a.lddst, L * a.lddst, kGridPos, 32 / kGridPos))
      return cudaErrorNotSupported;
    // P as [column group of 64][position][64 columns]: one box of 64 x 16 x 2 is a chunk's 16 rows
    if (!make_sw128_map3(&maps.p, a.shift.P, kUmmaCols, a.shift.max_pos, a.d / kUmmaCols, a.shift.ldp, kUmmaCols,
                         kGridPos, kChunkCols / kUmmaCols))
      return cudaErrorNotSupported;
  } else {
    if (!make_sw128_map3(&maps.z, a.zin, a.k, a.n, 1, a.ldzin, a.n * a.ldzin, kUmmaTile, 1))
      return cudaErrorNotSupported;
    if (!make_sw128_map3(&maps.out, a.dst, a.d, a.n, 1, a.lddst, a.n * a.lddst, 32, 1))
      return cudaErrorNotSupported;
    maps.p = maps.z;
  }
  if (!make_sw128_map(&maps.u, a.U, a.d, a.k, a.ldu, kUmmaCols)) return cudaErrorNotSupported;
  if (!make_sw128_map(&maps.u_wide, a.U, a.d, a.k <= 64 ? 64 : 128, a.ldu, kUmmaCols)) return cudaErrorNotSupported;
  if (a.k > 64) {
    if (has_e && has_p) return launch_umma_expand_one<2, true, true>(a, geo, maps, sm_count, stream);
    if (has_e) return launch_umma_expand_one<2, true, false>(a, geo, maps, sm_count, stream);
    if (has_p) return launch_umma_expand_one<2, false, true>(a, geo, maps, sm_count, stream);
    return launch_umma_expand_one<2, false, false>(a, geo, maps, sm_count, stream);
  }
  if (has_e && has_p) return launch_umma_expand_one<1, true, true>(a, geo, maps, sm_count, stream);
  if (has_e) return launch_umma_expand_one<1, true, false>(a, geo, maps, sm_count, stream);
  if (has_p) return launch_umma_expand_one<1, false, true>(a, geo, maps, sm_count, stream);
  return launch_umma_expand_one<1, false, false>(a, geo, maps, sm_count, stream);
}

namespace {
template <int NTP>
cudaError_t launch_tokens_ntp(const TokensArgs &t, const UmmaTokensMaps &maps, int grid, cudaStream_t stream) {
  auto kernel = codec_umma_tokens_kernel<NTP>;
  constexpr int smem = UmmaTokensConfig<NTP>::kSmemBytes;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  kernel<<<(unsigned)grid, kTokensThreads, smem, stream>>>(t, maps);
  return cudaGetLastError();
}
}  // namespace

cudaError_t launch_codec_umma_tokens(const __nv_bfloat16 *H, int64_t ldh, const __nv_bfloat16 *C, int64_t ldc,
                                     float *out, int64_t ldout, int64_t n, int32_t m, int32_t k,
                                     int sm_count, cudaStream_t stream) {
  if (H == nullptr || C == nullptr || out == nullptr || k > 128 || k < 1 || m < 1) return cudaErrorNotSupported;
  if (n < 4 * kUmmaTile || n > 0x7fffffffLL) return cudaErrorNotSupported;
  UmmaTokensMaps maps;
  if (!make_sw128_map(&maps.h, H, n, m, ldh, kUmmaCols)) return cudaErrorNotSupported;
  if (!make_sw128_map(&maps.c, C, n, k, ldc, kUmmaCols)) return cudaErrorNotSupported;
  if (!make_sw128_map(&maps.c_wide, C, n, k <= 64 ? 64 : 128, ldc, kUmmaCols)) return cudaErrorNotSupported;
  const int nblk = (m + kUmmaTile - 1) / kUmmaTile;
  const int64_t nstage = (n + kUmmaCols - 1) / kUmmaCols;
  // CTAs per column block: the count (up to 16) that fills whole waves of SMs best
  int64_t splits = 1;
  double best = 0.0;
  for (int64_t s = 1; s <= 16 && s <= nstage; ++s) {
    const int64_t ctas = nblk * s, waves = (ctas + sm_count - 1) / sm_count;
    const double fill = (double)ctas / (double)(waves * sm_count);
    if (fill > best + 1e-9) {
      best = fill;
      splits = s;
    }
  }
  TokensArgs t{};
  t.out = out;
  t.ldout = ldout;
  t.n = n;
  t.m = m;
  t.k = k;
  t.splits = (int32_t)splits;
  if (splits > 1) {
    cudaError_t e = cudaMemset2DAsync(out, (size_t)ldout * sizeof(float), 0, (size_t)k * sizeof(float), (size_t)m, stream);
    if (e != cudaSuccess) return e;
  }
  const int grid = (int)(nblk * splits);
  const int ntp = 2 * ((k + 15) / 16);
  if (ntp <= 2) return launch_tokens_ntp<2>(t, maps, grid, stream);
  if (ntp <= 4) return launch_tokens_ntp<4>(t, maps, grid, stream);
  if (ntp <= 6) return launch_tokens_ntp<6>(t, maps, grid, stream);
  if (ntp <= 8) return launch_tokens_ntp<8>(t, maps, grid, stream);
  if (ntp <= 12) return launch_tokens_ntp<12>(t, maps, grid, stream);
  return launch_tokens_ntp<16>(t, maps, grid, stream);
}

bool codec_mma_supports(int d, int k) {
  return d % 32 == 0 && (int64_t)d * 2 <= kZeroRowBytes && k >= 1 && k <= 128;
}

cudaError_t launch_codec_mma(const MmaArgs &a, bool shift, int mode, int sm_count,
                             cudaStream_t stream) {
  if (mode == kModeProject) {
    cudaError_t e = launch_codec_umma_project(a, shift, sm_count, stream);
    if (e != cudaErrorNotSupported) return e;
  }
  // wire rows and a second addend: only the tcgen05 projection takes them
  if (a.zout32 != nullptr || a.src2 != nullptr) return cudaErrorNotSupported;
  if (mode == (kModeProject | kModeExpand) && !shift) {
    cudaError_t e = launch_codec_umma_roundtrip(a, sm_count, stream);
    if (e != cudaErrorNotSupported) return e;
  }
  const int nt = (a.k + 7) / 8;
  // With few tokens per warp a second 16-row tile would be computed for nothing.
  const bool small = a.n <= (int64_t)sm_count * kMmaWarps * 16;
  if (small && nt <= 8) {
    // few rows per SM: the warps of a CTA share a row tile and split d
    return a.n > (int64_t)sm_count * 16 ? launch_dsplit<2>(a, shift, mode, nt, sm_count, stream)
                                        : launch_dsplit<1>(a, shift, mode, nt, sm_count, stream);
  }
  if (!small && mode == kModeExpand) {
    cudaError_t e = launch_codec_umma_expand(a, shift, sm_count, stream);
    if (e != cudaErrorNotSupported) return e;
    e = launch_expand64(a, shift, sm_count, stream);
    if (e != cudaErrorNotSupported) return e;
  }
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
