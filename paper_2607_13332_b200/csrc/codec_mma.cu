// Launchers of the mma.sync codec kernels and the dispatch between all tensor-core kernels.
#include "codec_mma.cuh"
#include "codec_mma_dsplit.cuh"
#include "codec_expand64.cuh"
#include "codec_umma.cuh"

#include "codec_mma_launch.h"

namespace ssn {
namespace {

// SSN_KVAR_E / SSN_KVAR_P bits of a launch whose kernel reads the rows of those tables
inline int shift_variant(const MmaArgs &a, bool shift) {
  return shift ? (a.shift.E != nullptr ? SSN_KVAR_E : 0) | (a.shift.P != nullptr ? SSN_KVAR_P : 0) : 0;
}

template <int NT, int MT, bool SHIFT, int MODE>
cudaError_t launch_one(const MmaArgs &a, int sm_count, cudaStream_t stream) {
  auto kernel = codec_mma_kernel<NT, MT, SHIFT, MODE>;
  constexpr int smem = kStages * UStageRing<NT>::kStageBytes;
  static std::atomic<uint64_t> configured{0};   // per instantiation, one bit per device
  if (smem > 48 * 1024) {
    cudaError_t e = allow_dynamic_smem(kernel, smem, configured);
    if (e != cudaSuccess) return e;
  }
  int64_t grid = (a.n + 15) / 16;
  if (grid > sm_count) grid = sm_count;
  kernel<<<(unsigned)grid, kMmaThreads, smem, stream>>>(a);
  note_kernel(SSN_KERNEL_MMA_SYNC, shift_variant(a, SHIFT) | (NT > 8 ? SSN_KVAR_WIDE : 0) | (MT == 2 ? SSN_KVAR_ALT : 0));
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
  static std::atomic<uint64_t> configured{0};   // per instantiation, one bit per device
  {
    cudaError_t e = allow_dynamic_smem(kernel, smem, configured);
    if (e != cudaSuccess) return e;
  }
  int64_t grid = (a.n + 16 * MT - 1) / (16 * MT);
  if (grid > sm_count) grid = sm_count;
  kernel<<<(unsigned)grid, kMmaThreads, smem, stream>>>(a);
  note_kernel(SSN_KERNEL_MMA_SYNC_DSPLIT, shift_variant(a, SHIFT) | (MT == 2 ? SSN_KVAR_ALT : 0));
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
  static std::atomic<uint64_t> configured{0};   // per instantiation, one bit per device
  if (smem > 48 * 1024) {
    cudaError_t e = allow_dynamic_smem(kernel, smem, configured);
    if (e != cudaSuccess) return e;
  }
  kernel<<<(unsigned)sm_count, kMmaThreads, smem, stream>>>(a);
  note_kernel(SSN_KERNEL_EXPAND64, shift_variant(a, SHIFT) | (PDEDUP ? SSN_KVAR_ALT : 0));
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

}  // namespace

namespace {
// One warp waits on a barrier that is initialised for one arrival and never gets it; the wait
// runs out after max_polls polls and the status bit is the only thing the kernel leaves behind.
__global__ void bounded_wait_selftest_kernel(int max_polls, int32_t *dev_status) {
  __shared__ __align__(8) uint64_t bar;
  const uint32_t b = smem_u32(&bar);
  if (threadIdx.x == 0) {
    mbar_init(b, 1);
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  __syncthreads();
  if (!mbar_wait(b, 0, max_polls) && threadIdx.x == 0) atomicOr(dev_status, SSN_DEV_TIMEOUT);
}
}  // namespace

cudaError_t launch_bounded_wait_selftest(int max_polls, int32_t *dev_status, cudaStream_t stream) {
  bounded_wait_selftest_kernel<<<1, 32, 0, stream>>>(max_polls, dev_status);
  return cudaGetLastError();
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
  // the row statistic: only the tcgen05 expansion produces it, at any token count it takes
  if (a.rowsumsq != nullptr)
    return mode == kModeExpand ? launch_codec_umma_expand(a, shift, sm_count, stream) : cudaErrorNotSupported;
  if (mode == (kModeProject | kModeExpand) && !shift) {
    cudaError_t e = launch_codec_umma_roundtrip(a, sm_count, stream);
    if (e != cudaErrorNotSupported) return e;
  }
  const int nt = (a.k + 7) / 8;
  // With few tokens per warp a second 16-row tile would be computed for nothing.
  const bool small = a.n <= (int64_t)sm_count * kMmaWarps * 16;
  // The tcgen05 expansion deals (tile, chunk) units to the SMs, so it fills the machine from 512
  // tokens on; measured against the few-rows kernel it wins wherever the output is 8 MB or more,
  // the model is wide or the rank needs the wide mma.sync tiles (16384 tokens, d = 4096: 48 us
  // against 127 us), and loses a few microseconds of set-up on the smallest outputs.
  if (small && mode == kModeExpand && (a.n * a.d >= (1 << 22) || a.d >= 2048 || nt > 8)) {
    cudaError_t e = launch_codec_umma_expand(a, shift, sm_count, stream);
    if (e != cudaErrorNotSupported) return e;
  }
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
