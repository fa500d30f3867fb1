// tcgen05 / TMA contraction over TOKENS (bf16 in, fp32 out, sm_100a), k <= 128:
//     G [m x k] = H^T C = sum_t H[t, :]^T C[t, :]          H: [n x m], C: [n x k]
// the weight-factor gradient of the reparameterized SSN (Eq. reparam and the chain rule quoted
// with it: dL/dZw = (dL/dW) U_k = H^T (dY U_k); C = dY U_k comes from the projection kernel).
//
// A work unit is a block of 128 columns of H (the M of the MMA) over a range of tokens (the K):
// per stage of 64 tokens the block arrives as an MN-major A operand (two TMA boxes of 64 tokens x
// 64 columns, as stored) and the 64 rows of C as an MN-major B operand (as stored); four
// tcgen05.mma (M=128, N=k rounded up to 16, K=16) accumulate in TMEM.  With fewer column blocks
// than SMs the tokens are split over several CTAs per block, which add their fp32 partial sums to
// the (zeroed) output with red.global; with one CTA per block the sums are stored.
//
//   warp 0  producer     warp 1  MMA issuer, owns the TMEM allocation     warps 2-5  epilogue
// Every wait is bounded; a wait that runs out sets the status word (when given) and the kernel
// still runs to its end.
#pragma once

#include "codec_umma.cuh"

namespace ssn {

constexpr int kTokensThreads = 192;

struct TokensArgs {
  float *out;        // [m x k] fp32, leading dimension ldout; zeroed by the caller when splits > 1
  int64_t ldout;
  int64_t n;         // tokens
  int32_t m, k;
  int32_t splits;    // CTAs per column block
  int32_t *dev_status;
};

struct UmmaTokensMaps {
  CUtensorMap h;             // H: boxes of 64 token rows x 64 columns
  CUtensorMap c, c_wide;     // C: boxes of 64 token rows x 64 coordinates (c_wide: see UmmaMaps)
};

template <int NTP>
struct UmmaTokensConfig {
  static_assert(NTP % 2 == 0 && NTP >= 2 && NTP <= 16, "N = 8*NTP must be a multiple of 16 up to 128");
  static constexpr int kN = NTP * 8;
  static constexpr int kKG = kN <= 64 ? 1 : 2;
  static constexpr int kABytes = 2 * kUmmaCols * 128;           // 64 tokens x 128 columns, two 64-column groups
  static constexpr int kBGroupBytes = kUmmaCols * 128;          // 64 tokens x 64 coordinates
  static constexpr int kStageBytes = kABytes + kKG * kBGroupBytes;
  static constexpr int kMaxSmem = 227 * 1024;
  static constexpr int kFit = (kMaxSmem - 1024 - 512) / kStageBytes;
  static constexpr int kStagesN = kFit < 8 ? kFit : 8;
  static constexpr int kTmemCols = kN <= 32 ? 32 : (kN <= 64 ? 64 : 128);
  static constexpr int kSmemBytes = 1024 + kStagesN * kStageBytes + (2 * kStagesN + 1) * 8 + 16;
};

template <int NTP>
__global__ void __launch_bounds__(kTokensThreads, 1)
codec_umma_tokens_kernel(const TokensArgs a, const __grid_constant__ UmmaTokensMaps maps) {
  using Cfg = UmmaTokensConfig<NTP>;
  constexpr int S = Cfg::kStagesN;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  // unit = (column block, token range)
  const int blk = (int)(blockIdx.x / a.splits), part = (int)(blockIdx.x % a.splits);
  const int64_t nstage_all = (a.n + kUmmaCols - 1) / kUmmaCols;
  const int64_t st_lo = (nstage_all * part) / a.splits, st_hi = (nstage_all * (part + 1)) / a.splits;
  const int col0 = blk * kUmmaTile;

  const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bars = smem0 + S * Cfg::kStageBytes;
  auto full_bar = [&](int s) { return bars + s * 8; };
  auto empty_bar = [&](int s) { return bars + (S + s) * 8; };
  const uint32_t acc_full_bar = bars + 2 * S * 8;
  const uint32_t tmem_slot = bars + (2 * S + 1) * 8;
  volatile uint32_t *tmem_slot_ptr =
      reinterpret_cast<volatile uint32_t *>(smem_raw + (tmem_slot - smem_u32(smem_raw)));

  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    mbar_init(acc_full_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(tmem_slot),
                 "r"(Cfg::kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
  const uint32_t tmem_base = *tmem_slot_ptr;
  bool dead = false;
  auto timed_out = [&]() {
    dead = true;
    if (a.dev_status) atomicOr(a.dev_status, SSN_DEV_TIMEOUT);
  };

  if (warp == 0) {
    // ------------------------------------------------------------------------- producer
    const uint64_t stream_in = l2_policy_evict_first();   // H is read once; C comes back for every column block
    int slot = 0;
    uint32_t parity = 1;
    for (int64_t st = st_lo; st < st_hi; ++st) {
      if (!dead && !mbar_wait(empty_bar(slot), parity)) timed_out();
      const uint32_t base = smem0 + (uint32_t)slot * Cfg::kStageBytes;
      if (lane == 0) {
        const int tok0 = (int)(st * kUmmaCols);
        mbar_expect_tx(full_bar(slot), Cfg::kStageBytes);
        tma_load_2d_hint(base, &maps.h, full_bar(slot), col0, tok0, stream_in);
        tma_load_2d_hint(base + Cfg::kABytes / 2, &maps.h, full_bar(slot), col0 + 64, tok0, stream_in);
        // the last box of C would read past its buffer through the wide map
#pragma unroll
        for (int g = 0; g < Cfg::kKG; ++g)
          tma_load_2d(base + Cfg::kABytes + g * Cfg::kBGroupBytes, st == nstage_all - 1 ? &maps.c : &maps.c_wide,
                      full_bar(slot), g * 64, tok0);
      }
      __syncwarp();
      if (++slot == S) {
        slot = 0;
        parity ^= 1u;
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      // both operands MN-major (bits 15 and 16)
      constexpr uint32_t idesc = umma_idesc(Cfg::kN, false) | (1u << 15);
      const uint64_t adesc0 = umma_desc(0, Cfg::kABytes / 2, 1024, 2);       // two 64-column groups 8 KB apart
      const uint64_t bdesc0 = umma_desc(0, Cfg::kBGroupBytes, 1024, 2);
      int slot = 0;
      uint32_t parity = 0;
      for (int64_t st = st_lo; st < st_hi; ++st) {
        if (!dead && !mbar_wait(full_bar(slot), parity)) timed_out();
        asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
        const uint32_t base = smem0 + (uint32_t)slot * Cfg::kStageBytes;
        const uint64_t ad = adesc0 + umma_desc_addr(base), bd = bdesc0 + umma_desc_addr(base + Cfg::kABytes);
#pragma unroll
        for (int j = 0; j < kUmmaCols / 16; ++j)   // a K step: 16 token rows = 2048 bytes of either tile
          umma_bf16(tmem_base, ad + j * 128, bd + j * 128, idesc, (st > st_lo || j > 0) ? 1u : 0u);
        umma_commit(empty_bar(slot));
        if (st == st_hi - 1) umma_commit(acc_full_bar);
        if (++slot == S) {
          slot = 0;
          parity ^= 1u;
        }
      }
    }
  } else {
    // ------------------------------------------------------------------------- epilogue
    const int quarter = warp & 3;   // TMEM lanes 32*quarter .. +31: columns col0 + 32*quarter + lane of H
    if (st_hi > st_lo) {
      if (!dead && !mbar_wait(acc_full_bar, 0)) timed_out();
      asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
      const int row = col0 + quarter * 32 + lane;          // row of the output = column of H
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16);
#pragma unroll
      for (int q = 0; q < Cfg::kN / 16; ++q) {
        uint32_t v[16];
        tmem_ld16(taddr + q * 16, v);
        asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
        if (row < a.m) {
          float *orow = a.out + (int64_t)row * a.ldout;
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const int col = q * 16 + i;
            if (col < a.k) {
              if (a.splits > 1)
                atomicAdd(orow + col, __uint_as_float(v[i]));
              else
                orow[col] = __uint_as_float(v[i]);
            }
          }
        }
      }
    }
  }

  asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem_base),
                 "r"(Cfg::kTmemCols) : "memory");
  }
}

}  // namespace ssn
