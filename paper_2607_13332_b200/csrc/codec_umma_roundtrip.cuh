// tcgen05 / TMA "project then expand" kernel of the SSN codec (bf16, sm_100a), k <= 128:
//     C = S U   (fp32, in tensor memory),   D = C U^T        S, D: [n x d]
// used for the weight re-projection W <- (W U) U^T of the original SSN (Sec. 4.1; S and D are
// then the same buffer) and for the projected gradient G U U^T.  A tile of 128 rows is read
// once and written once:
//
//   pass 1  as in the projection kernel: per stage one TMA box of S (128 rows x 64 columns) and
//           the 64 x k slice of U; four tcgen05.mma (M=128, N=k rounded up to 16, K=16) per
//           stage accumulate C in 64 TMEM columns.
//   split   the epilogue warps read C, optionally store it rounded to bf16 (the coordinates
//           output), and write it to shared memory as TWO bf16 operands C_hi + C_lo
//           (C_lo = bf16(C - C_hi)), so that the second product sees ~16 mantissa bits of the
//           fp32 coordinates.
//   pass 2  per chunk of 128 output columns: the 128 rows of U of the chunk arrive as a K-major
//           operand (one TMA load), 2*ceil(k/16) tcgen05.mma (M=128, N=128, K=16) accumulate
//           C_hi U^T + C_lo U^T into one of two 128-column accumulators; the epilogue warps
//           read it (one row per thread), round to bf16 into a swizzled staging slab and hand
//           32 rows x 64 columns at a time to a TMA store, which also clips the rows past n.
//
//   warp 0  pass-1 producer     warp 1  MMA issuer (pass 1: even stages; pass 2), owns the TMEM allocation
//   warps 2-5  epilogue (TMEM lanes 32*(warp%4) ..)     warp 6  pass-2 producer (U chunks)
//   warp 7  second pass-1 MMA issuer (odd stages, into the second half-accumulator of C)
//
// LEFT variant (W stored [d x m], the subspace on the rows: W <- U (U^T W)): a tile is a block of
// 128 COLUMNS of W over all d rows.  Pass 1 contracts over the rows, T^T = W_blk^T U, with the block
// as an MN-major A operand (boxes of 64 rows x 64 columns, as stored); pass 2 swaps the roles,
// D[128 rows x 128 columns] = U_chunk (A, K-major) x (C_hi + C_lo) (B, K-major), and the epilogue
// stores rows of W as before.
//
// Rows (columns) of a tile are only written after all of them have been read, and tiles are
// disjoint, so the call may be in place.  Every wait is bounded; a wait that runs out sets SSN_DEV_TIMEOUT
// (when the caller gave a status word) and the kernel still runs to its end.
#pragma once

#include "codec_mma_launch.h"
#include "codec_umma.cuh"

namespace ssn {

__device__ __forceinline__ void tma_store_2d(const CUtensorMap *map, uint32_t src, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];\n"
               ::"l"(map), "r"(src), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tma_store_2d_hint(const CUtensorMap *map, uint32_t src, int c0, int c1, uint64_t policy) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group.L2::cache_hint [%0, {%2, %3}], [%1], %4;\n"
               ::"l"(map), "r"(src), "r"(c0), "r"(c1), "l"(policy) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;\n" ::: "memory"); }
template <int N> __device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;\n" ::"n"(N) : "memory");
}
template <int N> __device__ __forceinline__ void bulk_wait() {
  asm volatile("cp.async.bulk.wait_group %0;\n" ::"n"(N) : "memory");
}

constexpr int kRoundTripThreads = 256;
constexpr int kChunkCols = 128;    // output columns per pass-2 accumulator

// Instruction descriptor with both operands K-major (pass 2).
__host__ __device__ constexpr uint32_t umma_idesc_kk(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kUmmaTile >> 4) << 24);
}

template <int NTP>
struct UmmaRoundTripConfig {
  static_assert(NTP % 2 == 0 && NTP >= 2 && NTP <= 16, "N = 8*NTP must be a multiple of 16 up to 128");
  static constexpr int kN = NTP * 8;
  static constexpr int kKG = kN <= 64 ? 1 : 2;                  // 64-coordinate groups (128-byte operand rows)
  static constexpr int kKSteps = kN / 16;                       // K steps of pass 2
  static constexpr int kTileBytes = kUmmaTile * 128;            // [128 rows x 128 B]
  static constexpr int kUGroupBytes = kUmmaCols * 128;          // pass 1: 64 rows of U, one 64-column group
  static constexpr int kUBytes = kKG * kUGroupBytes;
  static constexpr int kStageBytes = kTileBytes + kUBytes;
  static constexpr int kCBytes = kKG * kTileBytes;              // the coordinates as an operand: [128 x k]
  static constexpr int kU2Bytes = kKG * kChunkCols * 128;       // pass 2: 128 rows of U, K-major
  static constexpr int kU2Stages = 2;
  static constexpr int kStagingBytes = 4 * 2 * 4096;            // per epilogue warp two [32 x 128 B] slabs
  static constexpr int kFixedBytes = 2 * kCBytes + kU2Stages * kU2Bytes + kStagingBytes;
  static constexpr int kMaxSmem = 227 * 1024;
  static constexpr int kFit = (kMaxSmem - 1024 - 512 - kFixedBytes) / kStageBytes;
  static constexpr int kStagesN = kFit < 8 ? kFit : 8;
  static_assert(kStagesN >= 2, "no room for two stages");
  // TMEM columns: C in two halves (pass 1 has two issuing threads on alternate stages, as in the
  // projection kernel: one thread cannot issue as fast as the ring delivers), then two D buffers
  static constexpr int kAcc1Col = 0;
  static constexpr int kAcc1bCol = kN <= 64 ? 64 : 128;
  static constexpr int kDCol = kN <= 64 ? 128 : 256;
  static constexpr int kTmemCols = 512;
  static constexpr int kBars = 2 * kStagesN + 2 + 2 * kU2Stages + 4;
  static constexpr int kSmemBytes = 1024 + kStagesN * kStageBytes + kFixedBytes + kBars * 8 + 16;
};

constexpr int kRoundTripMaxMatrices = kMaxFusedMatrices;

// One launch takes up to kRoundTripMaxMatrices matrices [rows_i x d] (the output projections of
// a block, say): the tiles of all of them are dealt to the CTAs as one list.
struct UmmaRoundTripMaps {
  // U: 64 x 64 boxes (u_wide: see UmmaMaps); per matrix, S: boxes of 128 rows x 64 columns,
  // out: 32 rows x 64 columns
  CUtensorMap u, u_wide;
  CUtensorMap b1, b1_wide;   // the factor of pass 1 when it is not U (see MmaArgs::B1), else copies of u, u_wide
  CUtensorMap s[kRoundTripMaxMatrices], out[kRoundTripMaxMatrices];
  int64_t rows[kRoundTripMaxMatrices];
  int32_t tile_start[kRoundTripMaxMatrices + 1];   // first tile of each matrix; [count] = all tiles
  int32_t count;
};

template <int NTP, bool LEFT>
__global__ void __launch_bounds__(kRoundTripThreads, 1)
codec_umma_roundtrip_kernel(const MmaArgs a, const __grid_constant__ UmmaRoundTripMaps maps) {
  using Cfg = UmmaRoundTripConfig<NTP>;
  constexpr int S = Cfg::kStagesN, S2 = Cfg::kU2Stages;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");   // the next kernel may set up behind this one
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int nstage = (a.B1 != nullptr ? a.d1 : a.d) / kUmmaCols;   // pass 1 runs over the columns of the source
  const int nchunks = a.d / kChunkCols;
  const int64_t ntiles = maps.tile_start[maps.count];
  // tile -> matrix and first row (LEFT: first column)
  auto locate = [&](int64_t tile, int &w, int &row0) {
    w = 0;
    while (w + 1 < maps.count && tile >= maps.tile_start[w + 1]) ++w;
    row0 = (int)(tile - maps.tile_start[w]) * kUmmaTile;
  };

  const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t c_hi = smem0, c_lo = smem0 + Cfg::kCBytes;
  const uint32_t u2_ring = c_lo + Cfg::kCBytes;
  const uint32_t staging = u2_ring + S2 * Cfg::kU2Bytes;
  const uint32_t ring = staging + Cfg::kStagingBytes;
  const uint32_t bars = ring + S * Cfg::kStageBytes;
  auto full_bar = [&](int s) { return bars + s * 8; };
  auto empty_bar = [&](int s) { return bars + (S + s) * 8; };
  const uint32_t acc1_full_bar = bars + 2 * S * 8;
  const uint32_t c_ready_bar = bars + (2 * S + 1) * 8;
  auto u2_full_bar = [&](int s) { return bars + (2 * S + 2 + s) * 8; };
  auto u2_empty_bar = [&](int s) { return bars + (2 * S + 2 + S2 + s) * 8; };
  auto d_full_bar = [&](int b) { return bars + (2 * S + 2 + 2 * S2 + b) * 8; };
  auto d_empty_bar = [&](int b) { return bars + (2 * S + 2 + 2 * S2 + 2 + b) * 8; };
  const uint32_t tmem_slot = bars + Cfg::kBars * 8;
  volatile uint32_t *tmem_slot_ptr =
      reinterpret_cast<volatile uint32_t *>(smem_raw + (tmem_slot - smem_u32(smem_raw)));

  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    mbar_init(acc1_full_bar, 2);   // both pass-1 issuers
    mbar_init(c_ready_bar, 4);
    for (int s = 0; s < S2; ++s) {
      mbar_init(u2_full_bar(s), 1);
      mbar_init(u2_empty_bar(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(d_full_bar(b), 1);
      mbar_init(d_empty_bar(b), 4);
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
    // ------------------------------------------------------------------------- pass-1 producer
    const uint64_t stream_in = l2_policy_evict_first();   // every tile is read once
    int slot = 0;
    uint32_t parity = 1;   // a fresh "empty" barrier passes a wait on parity 1
    for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
      int w, row0;
      locate(tile, w, row0);
      for (int st = 0; st < nstage; ++st) {
        if (!dead && !mbar_wait(empty_bar(slot), parity)) timed_out();
        const uint32_t base = ring + (uint32_t)slot * Cfg::kStageBytes;
        if (lane == 0) {
          mbar_expect_tx(full_bar(slot), Cfg::kStageBytes);
          if (LEFT) {   // rows st*64.. of the column block: two boxes of 64 columns
            tma_load_2d_hint(base, &maps.s[w], full_bar(slot), row0, st * kUmmaCols, stream_in);
            tma_load_2d_hint(base + Cfg::kTileBytes / 2, &maps.s[w], full_bar(slot), row0 + 64, st * kUmmaCols, stream_in);
          } else {
            tma_load_2d_hint(base, &maps.s[w], full_bar(slot), st * kUmmaCols, row0, stream_in);
          }
#pragma unroll
          for (int ug = 0; ug < Cfg::kKG; ++ug)
            tma_load_2d(base + Cfg::kTileBytes + ug * Cfg::kUGroupBytes, st == nstage - 1 ? &maps.b1 : &maps.b1_wide,
                        full_bar(slot), ug * 64, st * kUmmaCols);
        }
        __syncwarp();
        if (++slot == S) {
          slot = 0;
          parity ^= 1u;
        }
      }
    }
  } else if (warp == 6) {
    // ------------------------------------------------------------------------- pass-2 producer
    int slot = 0;
    uint32_t parity = 1;
    for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
      for (int q = 0; q < nchunks; ++q) {
        if (!dead && !mbar_wait(u2_empty_bar(slot), parity)) timed_out();
        const uint32_t base = u2_ring + (uint32_t)slot * Cfg::kU2Bytes;
        if (lane == 0) {
          mbar_expect_tx(u2_full_bar(slot), Cfg::kU2Bytes);
#pragma unroll
          for (int kg = 0; kg < Cfg::kKG; ++kg) {   // per 64-coordinate group: 128 rows of 128 bytes
            tma_load_2d(base + kg * Cfg::kTileBytes, &maps.u_wide, u2_full_bar(slot), kg * 64, q * kChunkCols);
            tma_load_2d(base + kg * Cfg::kTileBytes + Cfg::kUGroupBytes, q == nchunks - 1 ? &maps.u : &maps.u_wide,
                        u2_full_bar(slot), kg * 64, q * kChunkCols + kUmmaCols);
          }
        }
        __syncwarp();
        if (++slot == S2) {
          slot = 0;
          parity ^= 1u;
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      // LEFT: the A operand of pass 1 is MN-major as well (bit 15)
      constexpr uint32_t idesc1 = umma_idesc(Cfg::kN, false) | (LEFT ? (1u << 15) : 0u);
      constexpr uint32_t idesc2 = umma_idesc_kk(kChunkCols);
      // descriptors without the start address, which is added per instruction (address / 16)
      const uint64_t kdesc = umma_desc(0, 16, 1024, 2);                 // K-major tile, rows of 128 B
      const uint64_t udesc = umma_desc(0, Cfg::kUGroupBytes, 1024, 2);  // U slice of pass 1 (MN-major)
      const uint64_t wdesc = umma_desc(0, Cfg::kTileBytes / 2, 1024, 2);  // LEFT: W block, two 64-column groups
      int slot = 0, uslot = 0;
      uint32_t parity = 0, uparity = 0;
      int64_t tcount = 0, ccount = 0;
      for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x, ++tcount) {
        const uint32_t acc1 = tmem_base + Cfg::kAcc1Col;
        for (int st = 0; st < nstage; ++st) {
          // both pass-1 issuers wait on every stage (a thread that skipped a barrier's phase could
          // take the phase before it for the one it wants); the odd stages are warp 7's
          if (!dead && !mbar_wait(full_bar(slot), parity)) timed_out();
          if ((st & 1) == 0) {
            asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
            const uint32_t base = ring + (uint32_t)slot * Cfg::kStageBytes;
            const uint64_t ad = (LEFT ? wdesc : kdesc) + umma_desc_addr(base), bd = udesc + umma_desc_addr(base + Cfg::kTileBytes);
#pragma unroll
            for (int j = 0; j < kUmmaCols / 16; ++j)   // a K step: 32 bytes of a K-major row, 16 rows of an MN-major tile
              umma_bf16(acc1, ad + j * (LEFT ? 128 : 2), bd + j * 128, idesc1, (st > 0 || j > 0) ? 1u : 0u);
            umma_commit(empty_bar(slot));
          }
          if (++slot == S) {
            slot = 0;
            parity ^= 1u;
          }
        }
        umma_commit(acc1_full_bar);
        if (!dead && !mbar_wait(c_ready_bar, (uint32_t)(tcount & 1))) timed_out();
        asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
        for (int q = 0; q < nchunks; ++q, ++ccount) {
          const int db = (int)(ccount & 1);
          if (!dead && !mbar_wait(d_empty_bar(db), (uint32_t)(((ccount >> 1) & 1) ^ 1))) timed_out();
          if (!dead && !mbar_wait(u2_full_bar(uslot), uparity)) timed_out();
          asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
          const uint32_t dacc = tmem_base + Cfg::kDCol + (uint32_t)db * kChunkCols;
          const uint64_t bd = kdesc + umma_desc_addr(u2_ring + (uint32_t)uslot * Cfg::kU2Bytes);
          const uint64_t hd = kdesc + umma_desc_addr(c_hi), ld = kdesc + umma_desc_addr(c_lo);
#pragma unroll
          for (int j = 0; j < Cfg::kKSteps; ++j) {
            // K step j: 32 bytes into the rows of 64-coordinate group j / 4
            const uint32_t ko = (uint32_t)(j >> 2) * (Cfg::kTileBytes >> 4) + (uint32_t)(j & 3) * 2;
            if (LEFT) {   // rows of U times the coordinates of the column block
              umma_bf16(dacc, bd + ko, hd + ko, idesc2, j > 0 ? 1u : 0u);
              umma_bf16(dacc, bd + ko, ld + ko, idesc2, 1u);
            } else {
              umma_bf16(dacc, hd + ko, bd + ko, idesc2, j > 0 ? 1u : 0u);
              umma_bf16(dacc, ld + ko, bd + ko, idesc2, 1u);
            }
          }
          umma_commit(u2_empty_bar(uslot));
          umma_commit(d_full_bar(db));
          if (++uslot == S2) {
            uslot = 0;
            uparity ^= 1u;
          }
        }
      }
    }
  } else if (warp == 7) {
    // ------------------------------------------------------------------------- second pass-1 issuer
    if (lane == 0) {
      constexpr uint32_t idesc1 = umma_idesc(Cfg::kN, false) | (LEFT ? (1u << 15) : 0u);
      const uint64_t kdesc = umma_desc(0, 16, 1024, 2);
      const uint64_t udesc = umma_desc(0, Cfg::kUGroupBytes, 1024, 2);
      const uint64_t wdesc = umma_desc(0, Cfg::kTileBytes / 2, 1024, 2);
      int slot = 0;
      uint32_t parity = 0;
      int64_t tcount = 0;
      for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x, ++tcount) {
        const uint32_t acc1b = tmem_base + Cfg::kAcc1bCol;
        for (int st = 0; st < nstage; ++st) {
          if (!dead && !mbar_wait(full_bar(slot), parity)) timed_out();
          if ((st & 1) == 1) {
            asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
            const uint32_t base = ring + (uint32_t)slot * Cfg::kStageBytes;
            const uint64_t ad = (LEFT ? wdesc : kdesc) + umma_desc_addr(base), bd = udesc + umma_desc_addr(base + Cfg::kTileBytes);
#pragma unroll
            for (int j = 0; j < kUmmaCols / 16; ++j)
              umma_bf16(acc1b, ad + j * (LEFT ? 128 : 2), bd + j * 128, idesc1, (st > 1 || j > 0) ? 1u : 0u);
            umma_commit(empty_bar(slot));
          }
          if (++slot == S) {
            slot = 0;
            parity ^= 1u;
          }
        }
        umma_commit(acc1_full_bar);
        // the epilogue must have read this tile's half before the next tile's MMAs overwrite it
        if (!dead && !mbar_wait(c_ready_bar, (uint32_t)(tcount & 1))) timed_out();
        asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
      }
    }
  } else if (warp >= 2 && warp < 6) {
    // ------------------------------------------------------------------------- epilogue
    const int quarter = warp & 3;   // the TMEM lanes this warp may read: 32*quarter .. +31
    const int r = quarter * 32 + lane;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const uint32_t slab0 = staging + (uint32_t)quarter * 8192;
    const uint64_t stream_out = l2_policy_evict_first();   // written once, not read again here
    const bool zvec = a.zout != nullptr && ((a.ldzout & 7) == 0) && ((reinterpret_cast<uintptr_t>(a.zout) & 15) == 0);
    int64_t tcount = 0, ccount = 0;
    for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x, ++tcount) {
      int w, row0;
      locate(tile, w, row0);
      const int64_t nrows = maps.rows[w];
      // ---- split: C (fp32, TMEM) -> C_hi, C_lo (bf16, shared memory)
      if (!dead && !mbar_wait(acc1_full_bar, (uint32_t)(tcount & 1))) timed_out();
      asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
      {
        uint32_t v[Cfg::kN / 16][16];
#pragma unroll
        for (int q = 0; q < Cfg::kN / 16; ++q) tmem_ld16(lane_addr + Cfg::kAcc1Col + q * 16, v[q]);
        asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
        if (nstage >= 2) {   // the odd stages' half (with a single stage it was never written)
#pragma unroll
          for (int q = 0; q < Cfg::kN / 16; ++q) {
            uint32_t w[16];
            tmem_ld16(lane_addr + Cfg::kAcc1bCol + q * 16, w);
            asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
#pragma unroll
            for (int i = 0; i < 16; ++i) v[q][i] = __float_as_uint(__uint_as_float(v[q][i]) + __uint_as_float(w[i]));
          }
        }
        const int64_t t = row0 + r;
#pragma unroll
        for (int c = 0; c < 8 * Cfg::kKG; ++c) {           // 16-byte pieces: 8 coordinates each
          uint32_t hi[4] = {0, 0, 0, 0}, lo[4] = {0, 0, 0, 0};
          if (c * 8 < Cfg::kN) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              // coordinates past k come from whatever followed U's columns in memory: drop them
              const float f0 = c * 8 + 2 * i < a.k ? __uint_as_float(v[c >> 1][(c & 1) * 8 + 2 * i]) : 0.f;
              const float f1 = c * 8 + 2 * i + 1 < a.k ? __uint_as_float(v[c >> 1][(c & 1) * 8 + 2 * i + 1]) : 0.f;
              const __nv_bfloat16 h0 = __float2bfloat16_rn(f0), h1 = __float2bfloat16_rn(f1);
              hi[i] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
              lo[i] = pack_bf16(f0 - __bfloat162float(h0), f1 - __bfloat162float(h1));
            }
            if (!LEFT && a.zout != nullptr && t < nrows) {
              __nv_bfloat16 *zrow = a.zout + t * a.ldzout;
              if (zvec && c * 8 + 8 <= a.k) {
                *reinterpret_cast<uint4 *>(zrow + c * 8) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
              } else {
#pragma unroll
                for (int i = 0; i < 8; ++i)
                  if (c * 8 + i < a.k)
                    zrow[c * 8 + i] = __ushort_as_bfloat16((unsigned short)(hi[i >> 1] >> ((i & 1) * 16)));
              }
            }
          }
          const uint32_t off = (uint32_t)(c >> 3) * Cfg::kTileBytes + (uint32_t)r * 128 +
                               (uint32_t)(((c & 7) ^ (r & 7)) << 4);
          asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};\n" ::"r"(c_hi + off), "r"(hi[0]), "r"(hi[1]),
                       "r"(hi[2]), "r"(hi[3]) : "memory");
          asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};\n" ::"r"(c_lo + off), "r"(lo[0]), "r"(lo[1]),
                       "r"(lo[2]), "r"(lo[3]) : "memory");
        }
      }
      asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
      asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(c_ready_bar);

      // ---- pass-2 chunks: D (fp32, TMEM) -> bf16 slabs -> TMA stores
      for (int q = 0; q < nchunks; ++q, ++ccount) {
        const int db = (int)(ccount & 1);
        if (!dead && !mbar_wait(d_full_bar(db), (uint32_t)((ccount >> 1) & 1))) timed_out();
        asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
#pragma unroll
        for (int g = 0; g < kChunkCols / 64; ++g) {
          uint32_t v[4][16];
#pragma unroll
          for (int i = 0; i < 4; ++i)
            tmem_ld16(lane_addr + Cfg::kDCol + (uint32_t)db * kChunkCols + g * 64 + i * 16, v[i]);
          asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
          if (g == kChunkCols / 64 - 1) {
            asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(d_empty_bar(db));
          }
          // the store that last read this slab (two stores ago) must be done reading it
          if (lane == 0) bulk_wait_read<1>();
          __syncwarp();
          const uint32_t slab = slab0 + (uint32_t)g * 4096;
          const uint32_t srow = slab + lane * 128;
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            const uint32_t *w = &v[c >> 1][(c & 1) * 8];
            const uint32_t o0 = pack_bf16(__uint_as_float(w[0]), __uint_as_float(w[1]));
            const uint32_t o1 = pack_bf16(__uint_as_float(w[2]), __uint_as_float(w[3]));
            const uint32_t o2 = pack_bf16(__uint_as_float(w[4]), __uint_as_float(w[5]));
            const uint32_t o3 = pack_bf16(__uint_as_float(w[6]), __uint_as_float(w[7]));
            asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};\n" ::"r"(srow + ((c ^ (lane & 7)) << 4)), "r"(o0),
                         "r"(o1), "r"(o2), "r"(o3) : "memory");
          }
          asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
          __syncwarp();
          if (lane == 0) {
            if (LEFT) {   // rows q*128 + 32*quarter .. of W, columns of this block
              if (row0 + g * 64 < nrows)
                tma_store_2d_hint(&maps.out[w], slab, row0 + g * 64, q * kChunkCols + quarter * 32, stream_out);
            } else if (row0 + quarter * 32 < nrows) {
              tma_store_2d_hint(&maps.out[w], slab, q * kChunkCols + g * 64, (int)(row0 + quarter * 32), stream_out);
            }
            bulk_commit();
          }
        }
      }
    }
    if (lane == 0) bulk_wait<0>();
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
