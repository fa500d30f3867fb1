// tcgen05 / TMA projection kernel of the SSN codec (bf16, sm_100a):
//     Z = X U - E[ids] U - P[pos] U        compress (SHIFT) / grad-project coefficients (!SHIFT)
//
// The subtraction of Eq. (ssn_compress) is moved through the contraction: the three products
// X U, E U and P U are accumulated in fp32 in tensor memory and combined in the epilogue.
// bf16 x bf16 products are exact in fp32, so the only rounding is fp32 accumulation, and no
// thread ever touches an element of X, E or P:
//
//   warp 0   producer.  Per stage (128 tokens x 64 columns) one TMA box load of X, one of the
//            P rows (positions of a tile are consecutive) and one of the 64 x k slice of U.
//   warps 1-3 (and 12)  MMA issuers: one thread each issues tcgen05.mma (M=128, N=k rounded up to
//            16, K=16) into its own accumulator and commits to the stage's "empty" barrier (the
//            tensor pipe retires one such instruction per ~87 clocks whatever its N).  In the
//            order X, X, E, E, P: an operand with two threads has them take alternate stages.
//            After a tile's last stage each commits to the accumulators' "full" barrier.  Warp 1
//            owns the TMEM allocation.
//   warps 4-7  epilogue: tcgen05.ld their 32 TMEM lanes (one token per thread), combine the
//            accumulators, round to bf16, store the Z rows; two sets of accumulators let a tile's
//            epilogue overlap the next tile's MMAs.
//   warps 8-11 (with E rows only)  gather the E rows of the tile: 8 lanes copy one 128-byte row
//            piece with cp.async straight into the swizzled tile, some stages ahead of the
//            barrier arrival that publishes them (an id outside the table points at a row of zeros).
//   A launch carries only the warps its roles need (8, 12 or 13).
//
// X, E and P tiles use the 128-byte swizzled K-major layout (rows of 128 bytes); U arrives as a
// 128-byte swizzled MN-major operand straight from its row-major storage.  Every wait is
// bounded; a wait that runs out sets SSN_DEV_TIMEOUT and the kernel still runs to its end.
#pragma once

#include <cuda.h>

#include "codec_mma.cuh"

namespace ssn {

constexpr int kUmmaTile = 128;     // tokens per tile (MMA M)
constexpr int kUmmaCols = 64;      // columns of X per stage (one 128-byte swizzle row)
constexpr int kWaitSpins = 1 << 22;

__device__ __forceinline__ void mbar_init(uint32_t bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Waits for the phase with the given parity; gives up (returns false) after `limit` polls.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int limit = kWaitSpins) {
  int spins = 0;
  while (!mbar_try_wait(bar, parity))
    if (++spins > limit) return false;
  return true;
}
// The same with cluster-scope acquire: the phase was completed by arrivals from the peer CTA
// that follow its writes into this CTA's shared memory.
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity) {
  int spins = 0;
  for (;;) {
    uint32_t ok;
    asm volatile(
        "{\n.reg .pred p;\n"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    if (ok) return true;
    if (++spins > kWaitSpins) return false;
  }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar,
                                            int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];\n"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
// L2 eviction policies for the copies below: evict_first for what streams through once (so that
// it does not push out what comes back), evict_last for the small operands every tile re-reads.
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;\n" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;\n" : "=l"(p));
  return p;
}
__device__ __forceinline__ void tma_load_2d_hint(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1,
                                                 uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cta.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;\n"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "l"(policy) : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap *map, uint32_t bar,
                                            int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];\n"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tma_gather4(uint32_t dst, const CUtensorMap *map, uint32_t bar,
                                            int c0, int r0, int r1, int r2, int r3) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cta.global.tile::gather4.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%3, %4, %5, %6, %7}], [%2];\n"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(r0), "r"(r1), "r"(r2), "r"(r3) : "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                          uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];\n"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
}

// Shared-memory operand descriptors (64-bit): start address, leading / stride byte offsets in
// 16-byte units, descriptor version 1, layout type in bits 61..63.
__device__ __forceinline__ uint64_t umma_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes,
                                              uint32_t layout_type) {
  return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | ((uint64_t)layout_type << 61);
}

// Start-address field of a descriptor (14 bits, address / 16).  The mask matters: in a cluster
// launch the shared-memory addresses of the CTAs of rank > 0 carry high bits, which would
// otherwise spill into the neighbouring fields when the address is added to a prebuilt descriptor.
__device__ __forceinline__ uint64_t umma_desc_addr(uint32_t addr) { return (uint64_t)((addr >> 4) & 0x3FFFu); }

// Instruction descriptor: fp32 accumulate, bf16 A (K-major, optionally negated) and bf16 B
// (MN-major), N and M encoded as N/8 and M/16.
__host__ __device__ constexpr uint32_t umma_idesc(int n, bool negate_a) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((negate_a ? 1u : 0u) << 13) | (1u << 16) |
         ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kUmmaTile >> 4) << 24);
}

// Last step of the projection epilogue for the token t whose KN accumulator values are in v:
// subtracts the terms that come from the prepared tables E U and P U (fp32) instead of an operand
// (sub_eu / sub_pu: that term has no operand in this launch), then stores the row of Z, in the
// storage dtype or as a wire row of fp32 words followed by the token id.
template <int KN>
__device__ __forceinline__ void store_projected_row(const MmaArgs &a, int64_t t, uint32_t (&v)[KN / 16][16],
                                                    bool sub_eu, bool sub_pu, bool vec) {
  auto subtract_row = [&](const float *row) {
    const bool vec4 = (reinterpret_cast<uintptr_t>(row) & 15) == 0;   // 128-bit loads inside the row
#pragma unroll
    for (int q = 0; q < KN / 16; ++q)
#pragma unroll
      for (int i = 0; i < 16; i += 4) {
        const int col = q * 16 + i;
        if (vec4 && col + 4 <= a.k) {
          const float4 w = __ldg(reinterpret_cast<const float4 *>(row + col));
          v[q][i] = __float_as_uint(__uint_as_float(v[q][i]) - w.x);
          v[q][i + 1] = __float_as_uint(__uint_as_float(v[q][i + 1]) - w.y);
          v[q][i + 2] = __float_as_uint(__uint_as_float(v[q][i + 2]) - w.z);
          v[q][i + 3] = __float_as_uint(__uint_as_float(v[q][i + 3]) - w.w);
        } else {
#pragma unroll
          for (int e = 0; e < 4; ++e)
            if (col + e < a.k)
              v[q][i + e] = __float_as_uint(__uint_as_float(v[q][i + e]) - __ldg(row + col + e));
        }
      }
  };
  if (sub_eu && a.shift.EU != nullptr) {
    const int64_t er = embedding_row(a.shift, t);
    if (er >= 0) subtract_row(a.shift.EU + er * a.shift.ldeu);
  }
  if (sub_pu && a.shift.PU != nullptr) {
    const int64_t pr = position_row(a.shift, t);
    if (pr >= 0) subtract_row(a.shift.PU + pr * a.shift.ldpu);
  }
  if (a.zout32 != nullptr) {   // wire row: fp32 coordinates, then the token id
    float *wrow = a.zout32 + t * a.ldzout32;
    const bool vec4 = ((a.ldzout32 & 3) == 0) && ((reinterpret_cast<uintptr_t>(a.zout32) & 15) == 0);
#pragma unroll
    for (int q = 0; q < KN / 16; ++q)
#pragma unroll
      for (int i = 0; i < 16; i += 4) {
        const int col = q * 16 + i;
        if (vec4 && col + 4 <= a.k) {
          *reinterpret_cast<uint4 *>(wrow + col) = make_uint4(v[q][i], v[q][i + 1], v[q][i + 2], v[q][i + 3]);
        } else {
#pragma unroll
          for (int e = 0; e < 4; ++e)
            if (col + e < a.k) wrow[col + e] = __uint_as_float(v[q][i + e]);
        }
      }
    if (a.wire_ids != nullptr) reinterpret_cast<int32_t *>(wrow)[a.k] = a.wire_ids[t];
    return;
  }
  __nv_bfloat16 *zrow = a.zout + t * a.ldzout;
#pragma unroll
  for (int q = 0; q < KN / 16; ++q) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int col = q * 16 + h * 8;
      if (vec && col + 8 <= a.k) {
        uint4 o;
        o.x = pack_bf16(__uint_as_float(v[q][h * 8 + 0]), __uint_as_float(v[q][h * 8 + 1]));
        o.y = pack_bf16(__uint_as_float(v[q][h * 8 + 2]), __uint_as_float(v[q][h * 8 + 3]));
        o.z = pack_bf16(__uint_as_float(v[q][h * 8 + 4]), __uint_as_float(v[q][h * 8 + 5]));
        o.w = pack_bf16(__uint_as_float(v[q][h * 8 + 6]), __uint_as_float(v[q][h * 8 + 7]));
        *reinterpret_cast<uint4 *>(zrow + col) = o;
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i)
          if (col + i < a.k) zrow[col + i] = __float2bfloat16_rn(__uint_as_float(v[q][h * 8 + i]));
      }
    }
  }
}

template <int NTP, bool HAS_E, bool HAS_P>
struct UmmaProjectConfig {
  static_assert(NTP % 2 == 0 && NTP >= 2 && NTP <= 16, "N = 8*NTP must be a multiple of 16 up to 128");
  static constexpr int kN = NTP * 8;
  static constexpr int kATileBytes = kUmmaTile * 128;               // 128 rows of 128 bytes
  static constexpr int kATiles = 1 + (HAS_E ? 1 : 0) + (HAS_P ? 1 : 0);
  static constexpr int kUGroups = kN <= 64 ? 1 : 2;                 // 64-column groups of U
  static constexpr int kUGroupBytes = kUmmaCols * 128;              // 64 rows of 128 bytes
  static constexpr int kUBytes = kUGroups * kUGroupBytes;
  static constexpr int kStageBytes = kATiles * kATileBytes + kUBytes;
  static constexpr int kTmaBytes = kStageBytes - (HAS_E ? kATileBytes : 0);
  static constexpr int kMaxSmem = 227 * 1024;
  static constexpr int kFit = (kMaxSmem - 1024 - 512) / kStageBytes;
  static constexpr int kStagesN = kFit < 10 ? kFit : 10;
  static_assert(kStagesN >= 2, "no room for two stages");
  // Stages between issuing a gather and publishing it.  Two less than the ring: with a lag of S - 1
  // the first stage is published only when every slot of the ring holds a pending gather, and the
  // issuers starve (E and P, S = 4: 151 us with a lag of 3, 133 us with 2, 145 us with 1).
  static constexpr int kGatherLag = kStagesN > 3 ? kStagesN - 2 : 1;
  static constexpr int kAccCols = kN <= 32 ? 32 : (kN <= 64 ? 64 : 128);   // TMEM columns per accumulator
  // MMA-issuing threads, each with an accumulator of its own.  One thread sustains a stage of
  // four MMAs, a wait and a commit per ~540 clocks, which is slower than the ring can deliver and
  // than the tensor pipe can run; so the X operand gets TWO threads that take alternate stages
  // (their accumulators are summed in the epilogue) wherever tensor memory has room for it, and
  // the E and P operands one thread each.
  // E gets the same split as X whenever it is present: the two halves are then combined as
  // (X0 - E0) + (X1 - E1), so that rows equal to their E rows still cancel exactly.
  // (With E and P the five accumulators would leave one buffer of tensor memory; measured, the split
  // gains nothing there: 135 against 133 us.)
  static constexpr int kXIssuers = (!HAS_E || (kN <= 64 && !HAS_P)) ? 2 : 1;
  static constexpr int kEIssuers = HAS_E ? kXIssuers : 0;
  static constexpr int kIssuers = kXIssuers + kEIssuers + (HAS_P ? 1 : 0);
  // Warps: 0 producer; 1-3 the first three issuers; 4-7 epilogue; with E rows 8-11 gather them and
  // warp 12 is the fourth issuer (E only, k <= 64).  A launch has only the warps its roles need, so
  // that the register budget of the epilogue (a whole accumulator row per thread) is not cut by
  // warps that would idle: 256 threads without E rows, 384 or 416 with them.
  static constexpr int kWarps = !HAS_E ? 8 : (kIssuers == 4 ? 13 : 12);
  static constexpr int kThreads = 32 * kWarps;
  static constexpr int kBufs = 2 * kIssuers * kAccCols <= 512 ? 2 : 1;   // accumulator sets (tiles in flight)
  // accumulator slots: kIssuers per buffer; a launch that shares the positional product keeps it
  // in buffer 0's slot of the P issuer (buffer 1's stays unused then)
  static constexpr int kAccSlots = kBufs * kIssuers;
  static constexpr int kTmemCols = (kAccSlots * kAccCols) <= 128 ? 128 : ((kAccSlots * kAccCols) <= 256 ? 256 : 512);
  static_assert(kAccSlots * kAccCols <= 512, "accumulators do not fit in tensor memory");
  static constexpr int kBarBytes = (2 * kStagesN + 6) * 8 + 16;
  static constexpr int kSmemBytes = 1024 + kStagesN * kStageBytes + kBarBytes;
};

// u describes U as it is ([d x k]: a 64-column box that reaches past column k is filled with
// zeros, which the TMA unit does slowly); u_wide claims 64 (128) columns per row with the same
// row pitch, so that a box never leaves the tensor: the columns past k then hold the start of
// the following rows, and feed only accumulator columns that are never stored.  u_wide is used
// for all stages but the last one of U, whose box would read past the end of the buffer.
// x2: a second matrix of rows to project with the same tiles (a.src2 != nullptr): the
// contraction then runs over the columns of x and, after them, over the columns of x2 against
// the same slices of U, i.e. Z = (X + X2) U with the sum never formed or rounded.
struct UmmaMaps {
  CUtensorMap x, p, u, u_wide, x2;
};

// Launches `kernel(a, maps)` as pairs of CTAs (clusters of two) that share their odd tile, one
// pair per two SMs; falls back to single CTAs where clusters cannot be scheduled.
template <typename Kernel>
cudaError_t launch_tile_pairs(Kernel kernel, int threads, int smem, const MmaArgs &a, const UmmaMaps &maps,
                              int sm_count, cudaStream_t stream) {
  const int64_t ntiles = (a.n + kUmmaTile - 1) / kUmmaTile;
  int64_t pairs = ntiles;   // with few tiles every pair has one and splits it over d
  if (pairs > sm_count / 2) pairs = sm_count / 2;
  if (pairs < 1)   // a single SM: no pairs
    return launch_dependent(kernel, (unsigned)(ntiles < sm_count ? ntiles : sm_count), threads, smem, stream, 1, a, maps);
  cudaError_t e = launch_dependent(kernel, (unsigned)(2 * pairs), threads, smem, stream, 2, a, maps);
  if (e == cudaSuccess) return e;
  // a device that cannot co-schedule the pairs: the same kernel without clusters
  cudaGetLastError();
  const int64_t grid = ntiles < sm_count ? ntiles : sm_count;
  return launch_dependent(kernel, (unsigned)grid, threads, smem, stream, 1, a, maps);
}

template <int NTP, bool HAS_E, bool HAS_P>
__global__ void __launch_bounds__((UmmaProjectConfig<NTP, HAS_E, HAS_P>::kThreads), 1)
codec_umma_project_kernel(const MmaArgs a, const __grid_constant__ UmmaMaps maps) {
  using Cfg = UmmaProjectConfig<NTP, HAS_E, HAS_P>;
  constexpr int kETile = 1, kPTile = HAS_E ? 2 : 1;   // order of the tiles inside a stage
  constexpr int S = Cfg::kStagesN;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");   // the next kernel may set up behind this one
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int nstage1 = a.d / kUmmaCols;                                  // stages of one matrix
  const int nstage = (!HAS_E && !HAS_P && a.src2 != nullptr) ? 2 * nstage1 : nstage1;
  const int64_t ntiles = (a.n + kUmmaTile - 1) / kUmmaTile;

  const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bars = smem0 + S * Cfg::kStageBytes;
  auto full_bar = [&](int s) { return bars + s * 8; };
  auto empty_bar = [&](int s) { return bars + (S + s) * 8; };
  auto acc_full_bar = [&](int b) { return bars + (2 * S + b) * 8; };
  auto acc_empty_bar = [&](int b) { return bars + (2 * S + 2 + b) * 8; };
  const uint32_t partial_ready_bar = bars + (2 * S + 4) * 8;   // pair schedule: the peer's partial sums have arrived
  const uint32_t ring_free_bar = bars + (2 * S + 5) * 8;       // pair schedule: the peer's stage ring may be overwritten
  const uint32_t tmem_slot = bars + (2 * S + 6) * 8;
  volatile uint32_t *tmem_slot_ptr =
      reinterpret_cast<volatile uint32_t *>(smem_raw + (tmem_slot - smem_u32(smem_raw)));

  // Tile schedule.  The CTAs run as pairs (clusters of two).  Pair c takes the tiles c, c + pairs,
  // c + 2 pairs, ...; its two CTAs take them alternately, and when their number is odd the last
  // tile is SPLIT: rank 0 contracts the first half of d, rank 1 the second half; then each sends
  // the fp32 partial sums of the 64 rows the OTHER finishes into that CTA's (by then idle) stage
  // ring through distributed shared memory, adds what it receives for its own 64 rows and stores
  // them.  512 tiles on 74 pairs are 3 or 3.5 tiles per CTA instead of 3 or 4.  A launch without
  // clusters is the same schedule with pairs of one CTA and no split.
  uint32_t cluster_size, cta_rank;
  asm volatile("mov.u32 %0, %%cluster_nctaid.x;\n" : "=r"(cluster_size));
  asm volatile("mov.u32 %0, %%cluster_ctarank;\n" : "=r"(cta_rank));
  const int64_t pairs = gridDim.x / cluster_size, pair = blockIdx.x / cluster_size;
  // Sharing the positional product.  Tiles at the same 128-position block of different sequences
  // subtract the same P U.  When the batch is made of whole sequences (a.pshare), the tiles are
  // enumerated position-block-major (L = block * sequences + sequence), every pair takes a
  // contiguous range of L, and a CTA keeps P U of its current block in a persistent accumulator:
  // the P rows are loaded and contracted only when the block changes.
  constexpr bool kCanShare = HAS_E && HAS_P && Cfg::kN <= 64;
  const bool pshare = kCanShare && a.pshare != 0;
  const int64_t nseq = pshare ? a.n / a.shift.seq_len : 1;
  const int64_t nblk = pshare ? a.shift.seq_len / kUmmaTile : 1;
  const int64_t l_lo = pshare ? (ntiles * pair) / pairs : 0;
  const int64_t pair_tiles = pshare ? (ntiles * (pair + 1)) / pairs - l_lo
                                    : (pair < ntiles ? (ntiles - pair + pairs - 1) / pairs : 0);
  const bool has_split = cluster_size == 2 && (pair_tiles & 1) && nstage >= 2;
  const int my_tiles = (int)(cluster_size == 2
                                 ? pair_tiles / 2 + (((pair_tiles & 1) && (has_split || cta_rank == 0)) ? 1 : 0)
                                 : pair_tiles);
  // i-th tile of this CTA: index, stage range, whether it is the split one
  auto block_of = [&](int64_t j) { return (l_lo + j) / nseq; };   // position block of the pair's j-th tile
  auto schedule = [&](int i, int64_t &tile, int &st_lo, int &st_hi, bool &split) {
    split = has_split && i == my_tiles - 1;
    const int64_t j = cluster_size == 2 ? (split ? pair_tiles - 1 : 2 * (int64_t)i + cta_rank) : i;
    if (pshare) {
      const int64_t L = l_lo + j, blk = L / nseq;
      tile = (L - blk * nseq) * nblk + blk;
    } else {
      tile = pair + j * pairs;
    }
    st_lo = split && cta_rank == 1 ? nstage / 2 : 0;
    st_hi = split && cta_rank == 0 ? nstage / 2 : nstage;
  };
  // What this CTA does about P U on its i-th tile, given the block it has cached (-1: none):
  // 0 = load and contract the P rows over its stage range, 1 = use the cached product,
  // 2 = nothing (rank 1 on the split tile when rank 0 subtracts its cached full product).
  auto p_action = [&](int i, bool split, int64_t &cached_blk) {
    if (!pshare) return 0;
    const int64_t j = cluster_size == 2 ? (split ? pair_tiles - 1 : 2 * (int64_t)i + cta_rank) : i;
    const int64_t blk = block_of(j);
    if (!split) {
      if (cached_blk == blk) return 1;
      cached_blk = blk;
      return 0;
    }
    // rank 0 reaches the split tile with the block of its previous tile (j - 2) cached
    const bool rank0_has = pair_tiles >= 3 && block_of(pair_tiles - 3) == blk;
    cached_blk = -1;
    return rank0_has ? (cta_rank == 0 ? 1 : 2) : 0;
  };
  constexpr int kPersistentAcc = Cfg::kIssuers - 1;   // TMEM slot of the cached P U: buffer 0's slot of the P issuer

  if (threadIdx.x == 0) {
    mbar_init(partial_ready_bar, 64);   // the threads of the peer's two sending warps
    mbar_init(ring_free_bar, 2);        // the peer's two receiving warps
    for (int s = 0; s < S; ++s) {
      mbar_init(full_bar(s), HAS_E ? 5 : 1);
      mbar_init(empty_bar(s), Cfg::kATiles);   // one commit per operand (the X threads take turns)
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(acc_full_bar(b), Cfg::kIssuers);
      mbar_init(acc_empty_bar(b), 4);
    }
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(tmem_slot),
                 "r"(Cfg::kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
  __syncthreads();
  // the peer's barriers must exist before anything arrives on them
  asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;\n" ::: "memory");
  asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
  const uint32_t tmem_base = *tmem_slot_ptr;
  // set-up done; nothing in global memory is touched before the kernel in front has completed
  asm volatile("griddepcontrol.wait;\n" ::: "memory");
  bool dead = false;
  auto timed_out = [&]() {
    dead = true;
    if (a.shift.dev_status) atomicOr(a.shift.dev_status, SSN_DEV_TIMEOUT);
  };

  if (warp == 0) {
    // ------------------------------------------------------------------------- producer
    // the rows to project pass through L2 once; the P rows come back for every sequence
    const uint64_t stream_in = l2_policy_evict_first(), keep = l2_policy_evict_last();
    int slot = 0;
    uint32_t parity = 1;   // a fresh "empty" barrier passes a wait on parity 1
    int64_t cached_blk = -1;
    for (int it = 0; it < my_tiles; ++it) {
      int64_t tile;
      int st_lo, st_hi;
      bool split;
      schedule(it, tile, st_lo, st_hi, split);
      const int64_t tok0 = tile * kUmmaTile;
      const int pos0 = HAS_P ? (int)(tok0 % a.shift.seq_len) : 0;
      const bool load_p = HAS_P && p_action(it, split, cached_blk) == 0;
      for (int st = st_lo; st < st_hi; ++st) {
        if (!dead && !mbar_wait(empty_bar(slot), parity)) timed_out();
        const uint32_t base = smem0 + (uint32_t)slot * Cfg::kStageBytes;
        const uint32_t bar = full_bar(slot);
        if (lane == 0) {
          mbar_expect_tx(bar, Cfg::kTmaBytes - (HAS_P && !load_p ? Cfg::kATileBytes : 0));
          const int su = st < nstage1 ? st : st - nstage1;   // slice of U; the second matrix starts over
          tma_load_2d_hint(base, st < nstage1 ? &maps.x : &maps.x2, bar, su * kUmmaCols, (int)tok0, stream_in);
          if (load_p) tma_load_2d_hint(base + kPTile * Cfg::kATileBytes, &maps.p, bar, st * kUmmaCols, pos0, keep);
#pragma unroll
          for (int ug = 0; ug < Cfg::kUGroups; ++ug)
            tma_load_2d(base + Cfg::kATiles * Cfg::kATileBytes + ug * Cfg::kUGroupBytes,
                        su == nstage1 - 1 ? &maps.u : &maps.u_wide, bar, ug * 64, su * kUmmaCols);
        }
        __syncwarp();
        if (++slot == S) {
          slot = 0;
          parity ^= 1u;
        }
      }
    }
  } else if (warp < 4 || warp == 12) {
    // ------------------------------------------------------------------------- MMA issuers
    // Issuer index `which` (= its accumulator slot in a buffer) and the A tile `opnd` it reads, in
    // the order X, X again (alternate stages) when kXIssuers == 2, E, E again when kEIssuers == 2,
    // P.  The epilogue combines X.U - E.U - P.U.  A stage is released when every operand's issuer
    // has committed.
    const int which = warp == 12 ? 3 : warp - 1;   // issuer index = its accumulator slot in a buffer
    const bool is_x = which < Cfg::kXIssuers, is_e = !is_x && which < Cfg::kXIssuers + Cfg::kEIssuers;
    const int opnd = is_x ? 0 : (is_e ? 1 : kPTile);
    const int half = is_x ? which : which - Cfg::kXIssuers;        // which of an operand's alternating threads
    const int halves = is_x ? Cfg::kXIssuers : (is_e ? Cfg::kEIssuers : 1);
    if (lane == 0 && which < Cfg::kIssuers) {
      constexpr uint32_t idesc = umma_idesc(Cfg::kN, false);
      // A tiles: K-major rows of 128 bytes, 8-row groups 1024 bytes apart.  U slice: MN-major,
      // 64-column groups kUGroupBytes apart, 8-row groups 1024 bytes apart.
      const uint64_t adesc0 = umma_desc(0, 16, 1024, 2), bdesc0 = umma_desc(0, Cfg::kUGroupBytes, 1024, 2);
      int slot = 0;
      uint32_t parity = 0;
      int64_t tcount = 0;
      int64_t cached_blk = -1;
      const bool p_issuer = HAS_P && opnd == kPTile;
      for (int it = 0; it < my_tiles; ++it, ++tcount) {
        int64_t tile;
        int st_lo, st_hi;
        bool split;
        schedule(it, tile, st_lo, st_hi, split);
        const int buf = (int)(tcount % Cfg::kBufs);
        const uint32_t acc_parity = (uint32_t)((tcount / Cfg::kBufs) & 1);
        if (!dead && !mbar_wait(acc_empty_bar(buf), acc_parity ^ 1u)) timed_out();
        // the P issuer of a sharing launch: contract only when the block changes, into the
        // persistent accumulator, once the previous tile's epilogue has read the old product
        const bool contract = !(p_issuer && p_action(it, split, cached_blk) != 0);
        if (p_issuer && pshare && contract && tcount > 0) {
          const int64_t prev = tcount - 1;
          if (!dead && !mbar_wait(acc_empty_bar((int)(prev % Cfg::kBufs)), (uint32_t)((prev / Cfg::kBufs) & 1)))
            timed_out();
        }
        asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
        const uint32_t d_tmem =
            tmem_base + (uint32_t)(p_issuer && pshare ? kPersistentAcc : buf * Cfg::kIssuers + which) * Cfg::kAccCols;
        for (int st = st_lo; st < st_hi; ++st) {
          // alternate stages when two threads share the one operand
          const bool mine = halves == 1 || ((st - st_lo) & 1) == half;
          // Every issuer waits on EVERY stage, its partner's too.  A parity wait tells apart only
          // the current phase of a barrier and the one before it: a thread that skipped its
          // partner's stages could reach a slot while the load of the slot's previous use (a
          // partner's stage, loads complete out of order) was still in flight, take that earlier
          // phase for its own, consume a half-written stage and arrive on "empty" once too often.
          if (!dead && !mbar_wait(full_bar(slot), parity)) timed_out();
          if (mine) {
            asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
            const uint32_t base = smem0 + (uint32_t)slot * Cfg::kStageBytes;
            // the start-address field (address / 16) is added to descriptors built once: a K step
            // is 32 bytes of an A row and 16 rows = 2048 bytes of the U slice
            const uint64_t adesc = adesc0 + umma_desc_addr(base + (uint32_t)opnd * Cfg::kATileBytes);
            const uint64_t bdesc = bdesc0 + umma_desc_addr(base + Cfg::kATiles * Cfg::kATileBytes);
            const int first_st = st_lo + (halves == 2 ? half : 0);   // this thread's first stage of the tile
            if (contract) {
#pragma unroll
              for (int j = 0; j < kUmmaCols / 16; ++j)
                umma_bf16(d_tmem, adesc + j * 2, bdesc + j * 128, idesc, (st > first_st || j > 0) ? 1u : 0u);
            }
            umma_commit(empty_bar(slot));
          }
          if (++slot == S) {
            slot = 0;
            parity ^= 1u;
          }
        }
        umma_commit(acc_full_bar(buf));   // arrives when every MMA this thread issued for the tile is done
      }
    }
  } else if (warp >= 8) {
    // ------------------------------------------------------------------------- E row gather
    if (HAS_E) {
      const int gw = warp - 8;                 // rows 32*gw .. 32*gw+31 of the tile
      const int piece = lane & 7, sub = lane >> 3;
      int slot = 0, pub_slot = 0, pending = 0;
      uint32_t parity = 1;
      auto publish = [&]() {                   // the oldest issued stage has landed
        asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(full_bar(pub_slot));
        if (++pub_slot == S) pub_slot = 0;
        --pending;
      };
      for (int it = 0; it < my_tiles; ++it) {
        int64_t tile;
        int st_lo, st_hi;
        bool split;
        schedule(it, tile, st_lo, st_hi, split);
        const int64_t tok0 = tile * kUmmaTile;
        const unsigned char *src[8];
        uint32_t dst[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int r = gw * 32 + i * 4 + sub;
          const int64_t t = tok0 + r;
          const int64_t er = t < a.n ? embedding_row(a.shift, t) : -1;
          src[i] = (er >= 0 ? reinterpret_cast<const unsigned char *>(
                                  static_cast<const __nv_bfloat16 *>(a.shift.E) + er * a.shift.lde)
                            : g_zero_row) + piece * 16;
          dst[i] = kETile * Cfg::kATileBytes + r * 128 + ((piece ^ (r & 7)) << 4);
        }
        for (int st = st_lo; st < st_hi; ++st) {
          if (!dead && !mbar_wait(empty_bar(slot), parity)) timed_out();
          const uint32_t base = smem0 + (uint32_t)slot * Cfg::kStageBytes;
#pragma unroll
          for (int i = 0; i < 8; ++i) cp_async16_cg(base + dst[i], src[i] + st * 128);
          cp_async_commit();
          if (++pending > Cfg::kGatherLag) {
            cp_async_wait<Cfg::kGatherLag>();
            publish();
          }
          if (++slot == S) {
            slot = 0;
            parity ^= 1u;
          }
        }
      }
      cp_async_wait<0>();
      while (pending > 0) publish();
    }
  } else {
    // ------------------------------------------------------------------------- epilogue
    const int quarter = warp & 3;   // the TMEM lanes this warp may read: 32*quarter .. +31
    int64_t tcount = 0;
    int64_t cached_blk = -1;
    const bool vec = ((a.ldzout & 7) == 0) && ((reinterpret_cast<uintptr_t>(a.zout) & 15) == 0);
    for (int it = 0; it < my_tiles; ++it, ++tcount) {
      int64_t tile;
      int st_lo, st_hi;
      bool split;
      schedule(it, tile, st_lo, st_hi, split);
      const int p_act = HAS_P ? p_action(it, split, cached_blk) : 0;
      const int buf = (int)(tcount % Cfg::kBufs);
      const uint32_t acc_parity = (uint32_t)((tcount / Cfg::kBufs) & 1);
      if (!dead && !mbar_wait(acc_full_bar(buf), acc_parity)) timed_out();
      asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
      const uint32_t taddr =
          tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * Cfg::kIssuers) * Cfg::kAccCols;
      uint32_t v[Cfg::kN / 16][16];
#pragma unroll
      for (int q = 0; q < Cfg::kN / 16; ++q) tmem_ld16(taddr + q * 16, v[q]);
      asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
      // Z = (X0 - E0) + (X1 - E1) - P.U: slot 0 is X0 (in v); E0 follows the X slots
      const bool two_halves = Cfg::kXIssuers == 2 && st_hi - st_lo >= 2;   // a single stage: the second threads had none
      auto combine = [&](uint32_t addr, int sign) {     // v += sign * accumulator at addr
#pragma unroll
        for (int q = 0; q < Cfg::kN / 16; ++q) {
          uint32_t w[16];
          tmem_ld16(addr + q * 16, w);
          asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
#pragma unroll
          for (int i = 0; i < 16; ++i)
            v[q][i] = __float_as_uint(sign > 0 ? __uint_as_float(v[q][i]) + __uint_as_float(w[i])
                                               : __uint_as_float(v[q][i]) - __uint_as_float(w[i]));
        }
      };
      if (HAS_E) combine(taddr + Cfg::kXIssuers * Cfg::kAccCols, -1);                    // X0 - E0
      if (two_halves) {
        if (Cfg::kEIssuers == 2) {                                                        // + (X1 - E1)
#pragma unroll
          for (int q = 0; q < Cfg::kN / 16; ++q) {
            uint32_t x1[16], e1[16];
            tmem_ld16(taddr + Cfg::kAccCols + q * 16, x1);
            tmem_ld16(taddr + (Cfg::kXIssuers + 1) * Cfg::kAccCols + q * 16, e1);
            asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
#pragma unroll
            for (int i = 0; i < 16; ++i)
              v[q][i] = __float_as_uint(__uint_as_float(v[q][i]) + (__uint_as_float(x1[i]) - __uint_as_float(e1[i])));
          }
        } else {
          combine(taddr + Cfg::kAccCols, +1);                                             // + X1
        }
      }
      if (HAS_P && p_act != 2)   // 2: the peer subtracts the whole product; a sharing launch keeps P.U persistent
        combine(pshare ? tmem_base + ((uint32_t)(quarter * 32) << 16) + kPersistentAcc * Cfg::kAccCols
                       : taddr + (Cfg::kIssuers - 1) * Cfg::kAccCols, -1);
      asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty_bar(buf));

      if (split) {
        // The split tile is the last one of both CTAs, and each finishes HALF of its rows: rank 0
        // the rows 0..63 (epilogue warps of quarters 0 and 1), rank 1 the rows 64..127.  A warp
        // either receives the peer's partial sums of its rows or sends its own to the peer.  Every
        // stage of a CTA's ring has been consumed once its accumulators are complete, so the ring
        // can carry the 64 rows it receives.
        const uint32_t row_off = (uint32_t)(quarter * 32 + lane) * (Cfg::kN * 4);
        const uint32_t peer = cta_rank ^ 1u;
        if ((uint32_t)(quarter >> 1) == cta_rank) {
          if (lane == 0) {   // this CTA's ring is idle: the peer may write into it
            uint32_t remote;
            asm volatile("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(remote) : "r"(ring_free_bar), "r"(peer));
            asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];\n" ::"r"(remote) : "memory");
          }
          if (!dead && !mbar_wait_cluster(partial_ready_bar, 0)) timed_out();
#pragma unroll
          for (int q = 0; q < Cfg::kN / 16; ++q)
#pragma unroll
            for (int i = 0; i < 16; i += 4) {
              float4 w;
              asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];\n"
                           : "=f"(w.x), "=f"(w.y), "=f"(w.z), "=f"(w.w) : "r"(smem0 + row_off + (q * 16 + i) * 4));
              v[q][i] = __float_as_uint(__uint_as_float(v[q][i]) + w.x);
              v[q][i + 1] = __float_as_uint(__uint_as_float(v[q][i + 1]) + w.y);
              v[q][i + 2] = __float_as_uint(__uint_as_float(v[q][i + 2]) + w.z);
              v[q][i + 3] = __float_as_uint(__uint_as_float(v[q][i + 3]) + w.w);
            }
        } else {
          if (!dead && !mbar_wait_cluster(ring_free_bar, 0)) timed_out();
          uint32_t remote_ring, remote_bar;
          asm volatile("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(remote_ring) : "r"(smem0 + row_off), "r"(peer));
          asm volatile("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(remote_bar) : "r"(partial_ready_bar), "r"(peer));
#pragma unroll
          for (int q = 0; q < Cfg::kN / 16; ++q)
#pragma unroll
            for (int i = 0; i < 16; i += 4)
              asm volatile("st.shared::cluster.v4.b32 [%0], {%1,%2,%3,%4};\n" ::"r"(remote_ring + (q * 16 + i) * 4),
                           "r"(v[q][i]), "r"(v[q][i + 1]), "r"(v[q][i + 2]), "r"(v[q][i + 3]) : "memory");
          asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];\n" ::"r"(remote_bar) : "memory");
          continue;   // the peer stores these rows
        }
      }

      const int64_t t = tile * kUmmaTile + quarter * 32 + lane;
      if (t < a.n) {
        store_projected_row<Cfg::kN>(a, t, v, !HAS_E, !HAS_P, vec);
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
  // neither CTA of a pair may leave while the other can still touch its shared memory
  asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;\n" ::: "memory");
}

}  // namespace ssn
