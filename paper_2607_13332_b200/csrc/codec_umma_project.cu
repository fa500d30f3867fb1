// Launcher of the tcgen05 projection kernel (see codec_umma.cuh).
#include "codec_umma.cuh"
#include "codec_tensor_maps.h"
#include "codec_mma_launch.h"

namespace ssn {
namespace {

template <int NTP, bool HAS_E, bool HAS_P>
cudaError_t launch_umma_one(const MmaArgs &a, const UmmaMaps &maps, int sm_count, cudaStream_t stream) {
  auto kernel = codec_umma_project_kernel<NTP, HAS_E, HAS_P>;
  constexpr int smem = UmmaProjectConfig<NTP, HAS_E, HAS_P>::kSmemBytes;
  static std::atomic<uint64_t> configured{0};   // per instantiation, one bit per device
  {
    cudaError_t e = allow_dynamic_smem(kernel, smem, configured);
    if (e != cudaSuccess) return e;
  }
  note_kernel(SSN_KERNEL_UMMA_PROJECT, (HAS_E ? SSN_KVAR_E : 0) | (HAS_P ? SSN_KVAR_P : 0) |
                                           (NTP > 8 ? SSN_KVAR_WIDE : 0) | (a.pshare ? SSN_KVAR_ALT : 0));
  return launch_tile_pairs(kernel, UmmaProjectConfig<NTP, HAS_E, HAS_P>::kThreads, smem, a, maps, sm_count, stream);
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

}  // namespace ssn
