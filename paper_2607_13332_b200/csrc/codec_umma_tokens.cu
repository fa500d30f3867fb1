// Launcher of the tcgen05 contraction over tokens (see codec_umma_tokens.cuh).
#include "codec_umma_tokens.cuh"
#include "codec_tensor_maps.h"
#include "codec_mma_launch.h"

namespace ssn {
namespace {
template <int NTP>
cudaError_t launch_tokens_ntp(const TokensArgs &t, const UmmaTokensMaps &maps, int grid, cudaStream_t stream) {
  auto kernel = codec_umma_tokens_kernel<NTP>;
  constexpr int smem = UmmaTokensConfig<NTP>::kSmemBytes;
  static std::atomic<uint64_t> configured{0};   // per instantiation, one bit per device
  {
    cudaError_t e = allow_dynamic_smem(kernel, smem, configured);
    if (e != cudaSuccess) return e;
  }
  kernel<<<(unsigned)grid, kTokensThreads, smem, stream>>>(t, maps);
  note_kernel(SSN_KERNEL_UMMA_TOKENS, NTP > 8 ? SSN_KVAR_WIDE : 0);
  return cudaGetLastError();
}
}  // namespace

cudaError_t launch_codec_umma_tokens(const __nv_bfloat16 *H, int64_t ldh, const __nv_bfloat16 *C, int64_t ldc,
                                     float *out, int64_t ldout, int64_t n, int32_t m, int32_t k,
                                     int32_t *dev_status, int sm_count, cudaStream_t stream) {
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
  t.dev_status = dev_status;
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

}  // namespace ssn
