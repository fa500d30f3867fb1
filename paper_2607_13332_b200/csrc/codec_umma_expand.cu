// Launcher of the tcgen05 expansion kernel (see codec_umma_expand.cuh).
#include "codec_umma_expand.cuh"
#include "codec_tensor_maps.h"
#include "codec_mma_launch.h"

namespace ssn {
namespace {

template <int KG, bool HAS_E, bool HAS_P, int PROWS = kGridPos>
cudaError_t launch_umma_expand_one(const MmaArgs &a, const ExpandGeometry &geo, const UmmaExpandMaps &maps,
                                   int sm_count, cudaStream_t stream) {
  auto kernel = codec_umma_expand_kernel<KG, HAS_E, HAS_P, PROWS>;
  constexpr int smem = UmmaExpandConfig<KG, HAS_E, HAS_P, PROWS>::kSmemBytes;
  static std::atomic<uint64_t> configured{0};   // per instantiation, one bit per device
  {
    cudaError_t e = allow_dynamic_smem(kernel, smem, configured);
    if (e != cudaSuccess) return e;
  }
  const int64_t units = geo.ntiles * (a.d / kChunkCols);     // (tile, chunk) pairs, dealt evenly
  int64_t grid = units < sm_count ? units : sm_count;
  const cudaError_t launched = launch_dependent(kernel, (unsigned)grid, kExpandThreads, smem, stream, 1, a, geo, maps);
  note_kernel(SSN_KERNEL_UMMA_EXPAND, (HAS_E ? SSN_KVAR_E : 0) | (HAS_P ? SSN_KVAR_P : 0) | (KG == 2 ? SSN_KVAR_WIDE : 0) |
                                          (geo.grid_mode ? SSN_KVAR_ALT : 0) | (a.rowsumsq != nullptr ? SSN_KVAR_ROWSUMSQ : 0) |
                                          (PROWS != kGridPos ? SSN_KVAR_FEWSEQ : 0) | (a.zin2 != nullptr ? SSN_KVAR_TWO_RUNS : 0));
  return launched;
}

}  // namespace

// Expansion (decompress) on tcgen05.  Returns cudaErrorNotSupported when the call should take the
// mma.sync kernel instead: k > 128, d not a multiple of 128, few tokens, no tensor map, or a
// position table with explicit positions / a batch that is not made of whole sequences that tile
// into g sequences x 128/g positions (g = 8: length a multiple of 16; else g = 4, 2, 1 with k <= 64).
cudaError_t launch_codec_umma_expand(const MmaArgs &a, bool shift, int sm_count, cudaStream_t stream) {
  if (a.zin == nullptr || a.dst == nullptr || a.src != nullptr) return cudaErrorNotSupported;
  if (a.d % kChunkCols != 0 || a.k > 128 || a.n < 4 * kUmmaTile || a.n > 0x7fffffffLL)
    return cudaErrorNotSupported;
  if (a.zin2 != nullptr && a.k > 64) return cudaErrorNotSupported;   // two runs share one 64-coordinate U chunk
  const bool has_e = shift && a.shift.E != nullptr, has_p = shift && a.shift.P != nullptr;
  ExpandGeometry geo{};
  geo.seq_len = a.shift.seq_len;
  if (has_p) {
    const int64_t L = a.shift.seq_len;
    if (a.shift.pos != nullptr || L < 1 || L > a.shift.max_pos || a.n % L != 0) return cudaErrorNotSupported;
    // tiles of gseqs sequences x gpos positions: 8 x 16 when the batch allows, else the widest
    // group of sequences that divides it (a small call of 1 to 6 sequences)
    const int64_t B = a.n / L;
    int gseqs = 0;
    for (int g = kGridSeqs; g >= 1 && gseqs == 0; g >>= 1)
      if (B % g == 0 && L % (kUmmaTile / g) == 0) gseqs = g;
    if (gseqs == 0 || (gseqs != kGridSeqs && a.k > 64)) return cudaErrorNotSupported;
    geo.grid_mode = 1;
    geo.gseqs = gseqs;
    geo.gpos = kUmmaTile / gseqs;
    geo.nsg = (int32_t)(B / gseqs);
    geo.ntiles = (int64_t)geo.nsg * (L / geo.gpos);
  } else {
    geo.grid_mode = 0;
    geo.nsg = 1;
    geo.ntiles = (a.n + kUmmaTile - 1) / kUmmaTile;
  }
  UmmaExpandMaps maps;
  if (geo.grid_mode) {
    const int64_t L = a.shift.seq_len, B = a.n / L;
    // a warp stores 32 rows of the tile: 32 / gpos whole sequences, or 32 positions of one
    const int out_pos = geo.gpos < 32 ? geo.gpos : 32;
    if (!make_sw128_map3(&maps.z, a.zin, a.k, L, B, a.ldzin, L * a.ldzin, geo.gpos, geo.gseqs))
      return cudaErrorNotSupported;
    maps.z2 = maps.z;
    if (a.zin2 != nullptr &&
        !make_sw128_map3(&maps.z2, a.zin2, a.k, L, B, a.ldzin, L * a.ldzin, geo.gpos, geo.gseqs))
      return cudaErrorNotSupported;
    if (!make_sw128_map3(&maps.out, a.dst, a.d, L, B, a.lddst, L * a.lddst, out_pos, 32 / out_pos))
      return cudaErrorNotSupported;
    // P as [column group of 64][position][64 columns]: one box of 64 x gpos x 2 is a chunk's rows
    if (!make_sw128_map3(&maps.p, a.shift.P, kUmmaCols, a.shift.max_pos, a.d / kUmmaCols, a.shift.ldp, kUmmaCols,
                         geo.gpos, kChunkCols / kUmmaCols))
      return cudaErrorNotSupported;
  } else {
    if (!make_sw128_map3(&maps.z, a.zin, a.k, a.n, 1, a.ldzin, a.n * a.ldzin, kUmmaTile, 1))
      return cudaErrorNotSupported;
    maps.z2 = maps.z;
    if (a.zin2 != nullptr && !make_sw128_map3(&maps.z2, a.zin2, a.k, a.n, 1, a.ldzin, a.n * a.ldzin, kUmmaTile, 1))
      return cudaErrorNotSupported;
    if (!make_sw128_map3(&maps.out, a.dst, a.d, a.n, 1, a.lddst, a.n * a.lddst, 32, 1))
      return cudaErrorNotSupported;
    maps.p = maps.z;
  }
  if (!make_sw128_map(&maps.u, a.U, a.d, a.k, a.ldu, kUmmaCols)) return cudaErrorNotSupported;
  if (!make_sw128_map(&maps.u_wide, a.U, a.d, a.k <= 64 ? 64 : 128, a.ldu, kUmmaCols)) return cudaErrorNotSupported;
  if (has_p && geo.gseqs != kGridSeqs) {   // few sequences: room for up to 128 rows of P per chunk
    if (has_e) return launch_umma_expand_one<1, true, true, kUmmaTile>(a, geo, maps, sm_count, stream);
    return launch_umma_expand_one<1, false, true, kUmmaTile>(a, geo, maps, sm_count, stream);
  }
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

}  // namespace ssn
