// Launchers of the tcgen05 project-then-expand kernel (see codec_umma_roundtrip.cuh).
#include "codec_umma_roundtrip.cuh"
#include "codec_tensor_maps.h"
#include "codec_mma_launch.h"

namespace ssn {
namespace {
template <int NTP, bool LEFT>
cudaError_t launch_roundtrip_ntp(const MmaArgs &a, const UmmaRoundTripMaps &maps, int sm_count, cudaStream_t stream) {
  auto kernel = codec_umma_roundtrip_kernel<NTP, LEFT>;
  constexpr int smem = UmmaRoundTripConfig<NTP>::kSmemBytes;
  static std::atomic<uint64_t> configured{0};   // per instantiation, one bit per device
  {
    cudaError_t e = allow_dynamic_smem(kernel, smem, configured);
    if (e != cudaSuccess) return e;
  }
  int64_t grid = maps.tile_start[maps.count];
  if (grid > sm_count) grid = sm_count;
  const cudaError_t launched = launch_dependent(kernel, (unsigned)grid, kRoundTripThreads, smem, stream, 1, a, maps);
  note_kernel(SSN_KERNEL_UMMA_ROUNDTRIP, (NTP > 8 ? SSN_KVAR_WIDE : 0) | (LEFT ? SSN_KVAR_ALT : 0));
  return launched;
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

}  // namespace ssn
