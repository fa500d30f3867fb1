// tcgen05 / TMA expansion kernel of the SSN codec (bf16, sm_100a), k <= 128 (KG = 1 or 2 groups
// of 64 coordinates, each a 128-byte operand row):
//     Xhat = Z U^T + E[ids] + P[pos]          decompress (receiver side of Eq. ssn_compress)
//
// A tile is 128 tokens, a chunk 128 output columns accumulated in 128 TMEM columns:
//     D  = Z_tile[128 x k] * (U rows of the chunk)^T     ceil(k/16) MMAs (M=128, N=128, K=16)
//     D += Sel[128 x 16]   * P_rows[16 x 128]            one MMA, see below
// and the epilogue adds the gathered E rows in fp32 before the single rounding to bf16.
//
// Positions.  With implicit positions (t mod seq_len) a tile is laid out as g sequences x 128/g
// consecutive positions (a 3-D TMA box), so it needs only 128/g rows of P, which enter the
// accumulator through a constant 0/1 selection matrix (row r selects position r mod 128/g):
// 1.0 * bf16 is exact and the sum is taken in fp32, so no thread touches P.  Batches of groups of
// 8 sequences take g = 8: 16 rows of P and ONE more MMA per chunk (PROWS = 16).  Other batches
// (the 1 to 6 sequences of a small call) take g = 4, 2 or 1 in the PROWS = 128 variant, which
// reserves shared memory for up to 128 rows of P per chunk and issues 128/(16 g) MMAs for them.
// Without P a tile is 128 consecutive tokens.
//
//   warp 0     producer: per tile the Z tile; per chunk the 128 rows of U (K-major operand)
//              and the 16 rows of P.
//   warp 1     MMA issuer (one thread), owns the TMEM allocation; two accumulators alternate.
//   warps 2-9  epilogue, two groups of four that take alternate chunks: tcgen05.ld one token
//              row per thread, add the E row piece from shared memory, round to bf16 into a
//              swizzled staging slab and hand 32 rows x 64 columns to a TMA store (which also
//              clips the rows past n).
//   warps 10-13  gather the E rows of the tile, 64 columns at a time, with cp.async into
//              swizzled stages (an id outside the table points at a row of zeros); the epilogue
//              forms the sum in place and the stage is the source of the TMA store; a stage
//              goes back to the gather warps as soon as the chunk's last store has read it.
//              The ring is handed over per quarter of a stage (32 rows): gather warp q fills the
//              rows that epilogue warp q of either group reads, and each quarter has its own
//              pair of barriers.
// L2: the output is stored with an evict_first policy and the P rows are loaded with evict_last,
// so that the streams do not push the 16 rows under a chunk out before the next group of
// sequences needs them.
// Every wait is bounded; a wait that runs out sets SSN_DEV_TIMEOUT and the kernel still ends.
#pragma once

#include "codec_umma_roundtrip.cuh"

namespace ssn {

constexpr int kExpandThreads = 448;
constexpr int kGatherWarps = 4;
constexpr int kGridSeqs = 8, kGridPos = 16;   // tile shape of the PROWS = 16 variant

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, uint32_t bar,
                                            int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];\n"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
// the same copy with an L2 eviction policy (createpolicy) for its lines
__device__ __forceinline__ void tma_load_3d_hint(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1,
                                                 int c2, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cta.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5}], [%2], %6;\n"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "l"(policy) : "memory");
}
__device__ __forceinline__ void tma_store_3d_hint(const CUtensorMap *map, uint32_t src, int c0, int c1, int c2,
                                                  uint64_t policy) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group.L2::cache_hint [%0, {%2, %3, %4}], [%1], %5;\n"
               ::"l"(map), "r"(src), "r"(c0), "r"(c1), "r"(c2), "l"(policy) : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap *map, uint32_t src, int c0, int c1, int c2) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];\n"
               ::"l"(map), "r"(src), "r"(c0), "r"(c1), "r"(c2) : "memory");
}

template <int KG, bool HAS_E, bool HAS_P, int PROWS = kGridPos>
struct UmmaExpandConfig {
  static_assert(PROWS == 16 || PROWS == 128, "rows of P per chunk the kernel reserves room for");
  static constexpr int kTileBytes = kUmmaTile * 128;            // [128 rows x 128 B]
  static constexpr int kZBytes = KG * kTileBytes;               // one Z tile: KG groups of 64 coordinates
  // With E and two coordinate groups the E ring would have 4 stages only: one Z tile instead of two
  // buys two more (the MMAs run up to two chunks ahead of the epilogue, which hides most of the
  // load of the next tile's Z).  With one group the ring is deep enough and the second tile pays.
  static constexpr int kZBufs = (HAS_E && KG == 2) ? 1 : 2;
  static constexpr int kU2Bytes = KG * kChunkCols * 128;        // 128 rows of U, K-major, KG groups
  static constexpr int kPBytes = HAS_P ? 2 * PROWS * 128 : 0;      // PROWS rows of P, two 64-column groups
  static constexpr int kSelBytes = HAS_P ? (PROWS <= 64 ? 1 : 2) * kTileBytes : 0;   // one tile per 64 positions
  static constexpr int kUStageBytes = kU2Bytes + kPBytes;
  // with E the shared memory is better spent on its ring; 128 rows of P per stage leave room for two
  static constexpr int kUStages = (HAS_E || KG == 2 || (HAS_P && PROWS > kGridPos)) ? 2 : 3;
  static constexpr int kEStageBytes = kTileBytes;               // E rows of 64 columns of a chunk
  // Without E the epilogue warps stage their output in two [32 x 128 B] slabs each; with E the
  // sum is formed in place in the E stage, which is then the source of the TMA store.
  static constexpr int kStagingBytes = HAS_E ? 0 : 8 * 2 * 4096;
  static constexpr int kFixedBytes =
      kZBufs * kZBytes + kSelBytes + kUStages * kUStageBytes + kStagingBytes;
  static constexpr int kMaxSmem = 227 * 1024;
  static constexpr int kEFit = (kMaxSmem - 1024 - 1024 - kFixedBytes) / kEStageBytes;
  static constexpr int kEStages = HAS_E ? (kEFit < 12 ? kEFit : 12) : 0;
  static_assert(!HAS_E || kEStages >= 4, "no room for the E ring");
  static constexpr int kDBufs = 2;                 // accumulators of 128 columns: one per epilogue group
  static constexpr int kTmemCols = 256;
  static constexpr int SE = HAS_E ? kEStages : 1;
  static constexpr int kBars = 4 + 2 * kUStages + 8 * SE + 2 * kDBufs;   // the E ring has a full and an empty barrier per stage and QUARTER
  static constexpr int kSmemBytes = 1024 + kFixedBytes + kEStages * kEStageBytes + kBars * 8 + 16;
  static_assert(kSmemBytes <= kMaxSmem, "the rings do not fit in shared memory");
};

struct UmmaExpandMaps {
  // z2: the second coordinate matrix of a two-run expansion (MmaArgs::zin2), else a copy of z
  CUtensorMap z2;
  // z: Z tile (box 64 x 128 rows, or 64 x 16 x 8); u / u_wide: 64 x 64 boxes of U (see UmmaMaps);
  // p: P viewed as [column group][row][64 columns], boxes of 64 x 16 rows x 2 groups; out: 64 columns x 32 rows (or 64 x 16 x 2)
  CUtensorMap z, u, u_wide, p, out;
};

struct ExpandGeometry {
  int32_t grid_mode;      // 1: tiles of gseqs sequences x gpos positions, 0: 128 consecutive tokens
  int32_t seq_len;
  int32_t nsg;            // groups of gseqs sequences
  int32_t gseqs, gpos;    // gseqs * gpos == 128
  int64_t ntiles;
};

template <int KG, bool HAS_E, bool HAS_P, int PROWS = kGridPos>
__global__ void __launch_bounds__(kExpandThreads, 1)
codec_umma_expand_kernel(const MmaArgs a, const ExpandGeometry geo, const __grid_constant__ UmmaExpandMaps maps) {
  using Cfg = UmmaExpandConfig<KG, HAS_E, HAS_P, PROWS>;
  // positions and sequences of a tile: fixed in the PROWS = 16 variant, the launch's otherwise
  const int gpos = PROWS == kGridPos ? kGridPos : geo.gpos, gseqs = PROWS == kGridPos ? kGridSeqs : geo.gseqs;
  constexpr int SU = Cfg::kUStages, SE = Cfg::SE;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");   // the next kernel may set up behind this one
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int nchunks = a.d / kChunkCols;
  const int ksteps = (a.k + 15) / 16;
  const int64_t ntiles = geo.ntiles;
  // Two coordinate matrices (head and remainder of fp32 wire rows) against the same U chunk: both
  // Z buffers hold one tile's pair, so the tiles are not double-buffered then (KG == 1 only).
  const bool two_runs = KG == 1 && a.zin2 != nullptr;
  const int zbufs = two_runs ? 1 : Cfg::kZBufs;

  const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t z_base = smem0;                                         // the Z tiles
  const uint32_t sel = z_base + Cfg::kZBufs * Cfg::kZBytes;              // selection matrix (HAS_P)
  const uint32_t u_ring = sel + Cfg::kSelBytes;
  const uint32_t staging = u_ring + SU * Cfg::kUStageBytes;
  const uint32_t e_ring = staging + Cfg::kStagingBytes;
  const uint32_t bars = e_ring + Cfg::kEStages * Cfg::kEStageBytes;
  auto z_full_bar = [&](int b) { return bars + b * 8; };
  auto z_empty_bar = [&](int b) { return bars + (2 + b) * 8; };
  auto u_full_bar = [&](int s) { return bars + (4 + s) * 8; };
  auto u_empty_bar = [&](int s) { return bars + (4 + SU + s) * 8; };
  // The E ring is handed over per QUARTER of a stage (32 rows: one gather warp fills them, one
  // epilogue warp of either group consumes them), so that a late row holds up only its own quarter.
  auto e_full_bar = [&](int s, int q) { return bars + (4 + 2 * SU + 4 * s + q) * 8; };
  auto e_empty_bar = [&](int s, int q) { return bars + (4 + 2 * SU + 4 * SE + 4 * s + q) * 8; };
  auto d_full_bar = [&](int b) { return bars + (4 + 2 * SU + 8 * SE + b) * 8; };
  auto d_empty_bar = [&](int b) { return bars + (4 + 2 * SU + 8 * SE + Cfg::kDBufs + b) * 8; };
  const uint32_t tmem_slot = bars + Cfg::kBars * 8;
  volatile uint32_t *tmem_slot_ptr =
      reinterpret_cast<volatile uint32_t *>(smem_raw + (tmem_slot - smem_u32(smem_raw)));

  if (HAS_P) {
    // Sel[r][j] = 1 for j == r mod gpos (K-major, 128-byte rows of 64 positions, swizzled; a second
    // tile holds positions 64..127); only K = gpos is read
    for (uint32_t i = threadIdx.x; i < Cfg::kSelBytes / 16; i += blockDim.x) {
      const uint32_t tile = i / (Cfg::kTileBytes / 16), ii = i % (Cfg::kTileBytes / 16);
      const uint32_t r = ii >> 3, c = ii & 7;     // row, logical 16-byte piece
      uint4 v = make_uint4(0, 0, 0, 0);
      const uint32_t j = r % (uint32_t)gpos;      // the position row r selects
      if (tile == (j >> 6) && c == ((j & 63) >> 3)) {
        const uint32_t e = j & 7, word = 0x3F80u << ((e & 1) * 16);
        if ((e >> 1) == 0) v.x = word;
        if ((e >> 1) == 1) v.y = word;
        if ((e >> 1) == 2) v.z = word;
        if ((e >> 1) == 3) v.w = word;
      }
      const uint32_t off = tile * Cfg::kTileBytes + r * 128 + ((c ^ (r & 7)) << 4);
      *reinterpret_cast<uint4 *>(smem_raw + (sel - smem_u32(smem_raw)) + off) = v;
    }
    asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
  }
  if (threadIdx.x == 0) {
    for (int b = 0; b < 2; ++b) {
      mbar_init(z_full_bar(b), 1);
      mbar_init(z_empty_bar(b), 1);
    }
    for (int b = 0; b < Cfg::kDBufs; ++b) {
      mbar_init(d_full_bar(b), 1);
      mbar_init(d_empty_bar(b), 4);
    }
    for (int s = 0; s < SU; ++s) {
      mbar_init(u_full_bar(s), 1);
      mbar_init(u_empty_bar(s), 1);
    }
    for (int s = 0; s < SE; ++s) {
      for (int q = 0; q < 4; ++q) {
        mbar_init(e_full_bar(s, q), 32);             // one arrival per thread of the quarter's gather warp
        mbar_init(e_empty_bar(s, q), 1);             // the epilogue warp that consumed the quarter
      }
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
  // Work is dealt in units of (tile, chunk): chunks are independent output columns, so a CTA takes
  // a contiguous, balanced range of units and may start and end in the middle of a tile.
  const int64_t units = ntiles * nchunks;
  const int64_t u_lo = (units * blockIdx.x) / gridDim.x, u_hi = (units * (blockIdx.x + 1)) / gridDim.x;
  const int64_t tile_lo = u_lo / nchunks, tile_hi = u_hi > u_lo ? (u_hi - 1) / nchunks : tile_lo - 1;
  auto chunk_range = [&](int64_t tile, int &q0, int &q1) {
    q0 = tile == tile_lo ? (int)(u_lo - tile_lo * nchunks) : 0;
    q1 = tile == tile_hi ? (int)(u_hi - tile_hi * nchunks) : nchunks;
  };
  // tile -> TMA coordinates (row coordinate, sequence coordinate) of its first token
  auto tile_coords = [&](int64_t tile, int &c1, int &c2) {
    if (geo.grid_mode) {
      const int64_t pb = tile / geo.nsg;
      c1 = (int)pb * gpos;
      c2 = (int)(tile - pb * geo.nsg) * gseqs;
    } else {
      c1 = (int)(tile * kUmmaTile);
      c2 = 0;
    }
  };

  if (warp == 0) {
    // ------------------------------------------------------------------------- producer
    // The output streams through L2 once (and E mostly too) while the 16 rows of P under a chunk
    // come back for every group of sequences: without a hint they are evicted in between and every
    // chunk waits for DRAM (decompress with P: 172 -> 149 us with this hint alone).
    const uint64_t keep = l2_policy_evict_last();
    int slot = 0;
    uint32_t parity = 1;
    int64_t tcount = 0;
    for (int64_t tile = tile_lo; tile <= tile_hi; ++tile, ++tcount) {
      int c1, c2;
      tile_coords(tile, c1, c2);
      const int zb = (int)(tcount % zbufs);
      if (!dead && !mbar_wait(z_empty_bar(zb), (uint32_t)(((tcount / zbufs) & 1) ^ 1))) timed_out();
      if (lane == 0) {
        mbar_expect_tx(z_full_bar(zb), two_runs ? 2 * Cfg::kTileBytes : Cfg::kZBytes);
#pragma unroll
        for (int kg = 0; kg < KG; ++kg)
          tma_load_3d(z_base + zb * Cfg::kZBytes + kg * Cfg::kTileBytes, &maps.z, z_full_bar(zb), kg * 64, c1, c2);
        if (two_runs) tma_load_3d(z_base + Cfg::kTileBytes, &maps.z2, z_full_bar(zb), 0, c1, c2);
      }
      int q0, q1;
      chunk_range(tile, q0, q1);
      for (int q = q0; q < q1; ++q) {
        if (!dead && !mbar_wait(u_empty_bar(slot), parity)) timed_out();
        const uint32_t base = u_ring + (uint32_t)slot * Cfg::kUStageBytes;
        if (lane == 0) {
          mbar_expect_tx(u_full_bar(slot), Cfg::kU2Bytes + (HAS_P ? 2 * gpos * 128 : 0));
#pragma unroll
          for (int kg = 0; kg < KG; ++kg) {   // per group of 64 coordinates: 128 rows of 128 bytes
            tma_load_2d(base + kg * Cfg::kTileBytes, &maps.u_wide, u_full_bar(slot), kg * 64, q * kChunkCols);
            tma_load_2d(base + kg * Cfg::kTileBytes + 8192, q == nchunks - 1 ? &maps.u : &maps.u_wide,
                        u_full_bar(slot), kg * 64, q * kChunkCols + 64);
          }
          if (HAS_P) {
            // both 64-column groups of the 16 P rows in one copy (a 3-D view of P)
            tma_load_3d_hint(base + Cfg::kU2Bytes, &maps.p, u_full_bar(slot), 0, c1, q * (kChunkCols / kUmmaCols),
                             keep);
          }
        }
        __syncwarp();
        if (++slot == SU) {
          slot = 0;
          parity ^= 1u;
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_kk = umma_idesc_kk(kChunkCols);            // Z tile x U chunk, both K-major
      constexpr uint32_t idesc_kmn = umma_idesc(kChunkCols, false);       // Sel (K-major) x P rows (MN-major)
      const uint64_t kdesc = umma_desc(0, 16, 1024, 2);
      const uint64_t pdesc = umma_desc(0, (uint32_t)gpos * 128, 1024, 2); // 64-column groups gpos rows apart
      const uint64_t seld = kdesc + umma_desc_addr(sel);
      int slot = 0;
      uint32_t parity = 0;
      int64_t tcount = 0, ccount = 0;
      for (int64_t tile = tile_lo; tile <= tile_hi; ++tile, ++tcount) {
        const int zb = (int)(tcount % zbufs);
        if (!dead && !mbar_wait(z_full_bar(zb), (uint32_t)((tcount / zbufs) & 1))) timed_out();
        const uint64_t zd = kdesc + umma_desc_addr(z_base + zb * Cfg::kZBytes);
        const uint64_t zd2 = kdesc + umma_desc_addr(z_base + Cfg::kTileBytes);
        int q0, q1;
        chunk_range(tile, q0, q1);
        for (int q = q0; q < q1; ++q, ++ccount) {
          const int db = (int)(ccount % Cfg::kDBufs);
          if (!dead && !mbar_wait(d_empty_bar(db), (uint32_t)(((ccount / Cfg::kDBufs) & 1) ^ 1))) timed_out();
          if (!dead && !mbar_wait(u_full_bar(slot), parity)) timed_out();
          asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
          const uint32_t base = u_ring + (uint32_t)slot * Cfg::kUStageBytes;
          const uint32_t dacc = tmem_base + (uint32_t)db * kChunkCols;
          const uint64_t bd = kdesc + umma_desc_addr(base);
          for (int j = 0; j < ksteps; ++j) {   // K step j: 32 bytes into the rows of group j / 4
            const uint32_t ko = (uint32_t)(j >> 2) * (Cfg::kTileBytes >> 4) + (uint32_t)(j & 3) * 2;
            umma_bf16(dacc, zd + ko, bd + ko, idesc_kk, j > 0 ? 1u : 0u);
          }
          if (two_runs)
            for (int j = 0; j < ksteps; ++j) umma_bf16(dacc, zd2 + (uint32_t)j * 2, bd + (uint32_t)j * 2, idesc_kk, 1u);
          if (HAS_P) {
            // K step j: 16 positions = 32 bytes of a Sel row (a second tile from position 64 on)
            // and 16 rows = 2048 bytes of the P operand
            const uint64_t pd = pdesc + umma_desc_addr(base + Cfg::kU2Bytes);
            for (int j = 0; j < gpos / 16; ++j)
              umma_bf16(dacc, seld + (uint32_t)(j >> 2) * (Cfg::kTileBytes >> 4) + (uint32_t)(j & 3) * 2,
                        pd + (uint32_t)j * 128, idesc_kmn, 1u);
          }
          umma_commit(u_empty_bar(slot));
          umma_commit(d_full_bar(db));
          if (q == q1 - 1) umma_commit(z_empty_bar(zb));
          if (++slot == SU) {
            slot = 0;
            parity ^= 1u;
          }
        }
      }
    }
  } else if (warp >= 10) {
    // ------------------------------------------------------------------------- E row gather
    // 8 lanes copy one 128-byte row piece with cp.async straight into the swizzled stage; the
    // stage's "full" barrier counts one arrival per gather thread, made by the hardware when
    // that thread's copies have landed, so nothing waits between issuing stages.
    if (HAS_E) {
      const int gw = warp - 10;                // rows 32*gw .. 32*gw+31 of the tile
      const int piece = lane & 7, sub = lane >> 3;
      int slot = 0;
      uint32_t parity = 1;
      for (int64_t tile = tile_lo; tile <= tile_hi; ++tile) {
        int c1, c2;
        tile_coords(tile, c1, c2);
        const unsigned char *src[8];
        uint32_t dst[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int r = gw * 32 + i * 4 + sub;
          const int64_t t = geo.grid_mode ? (int64_t)(c2 + r / gpos) * geo.seq_len + c1 + r % gpos
                                          : (int64_t)c1 + r;
          const int64_t er = t < a.n ? embedding_row(a.shift, t) : -1;
          src[i] = (er >= 0 ? reinterpret_cast<const unsigned char *>(
                                  static_cast<const __nv_bfloat16 *>(a.shift.E) + er * a.shift.lde)
                            : g_zero_row) + piece * 16;
          dst[i] = r * 128 + ((piece ^ (r & 7)) << 4);
        }
        int q0, q1;
        chunk_range(tile, q0, q1);
        for (int qg = 2 * q0; qg < 2 * q1; ++qg) {     // 64-column groups of the row
          if (!dead && !mbar_wait(e_empty_bar(slot, gw), parity)) timed_out();
          const uint32_t base = e_ring + (uint32_t)slot * Cfg::kEStageBytes;
#pragma unroll
          for (int i = 0; i < 8; ++i) cp_async16_cg(base + dst[i], src[i] + qg * 128);
          asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];\n" ::"r"(e_full_bar(slot, gw)) : "memory");
          if (++slot == SE) {
            slot = 0;
            parity ^= 1u;
          }
        }
      }
      cp_async_commit();
      cp_async_wait<0>();
    }
  } else {
    // ------------------------------------------------------------------------- epilogue
    const int quarter = warp & 3;                 // TMEM lanes 32*quarter .. +31
    const int group = warp >= 6 ? 1 : 0;          // takes the chunks with (chunk counter & 1) == group
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const uint32_t slab0 = staging + (uint32_t)(group * 4 + quarter) * 8192;   // !HAS_E: two slabs
    int64_t ccount = 0;
    int held = -1;                                // E stage whose store may still be reading it
    const uint64_t stream_out = l2_policy_evict_first();   // the output is written once and not read here
    for (int64_t tile = tile_lo; tile <= tile_hi; ++tile) {
      int c1, c2;
      tile_coords(tile, c1, c2);
      // first token row of this warp's 32 rows, as TMA store coordinates
      // (32 rows are 32 / gpos whole sequences, or 32 positions of one sequence when gpos >= 32)
      const int s1 = geo.grid_mode ? c1 + (quarter * 32) % gpos : c1 + quarter * 32;
      const int s2 = geo.grid_mode ? c2 + (quarter * 32) / gpos : 0;
      const bool rows_live = geo.grid_mode || (int64_t)s1 < a.n;
      // this thread's token (row quarter * 32 + lane of the tile), for the row statistic
      const int trow = quarter * 32 + lane;
      const int64_t tok = geo.grid_mode ? (int64_t)(c2 + trow / gpos) * geo.seq_len + c1 + trow % gpos
                                        : (int64_t)c1 + trow;
      int q0, q1;
      chunk_range(tile, q0, q1);
      for (int q = q0; q < q1; ++q, ++ccount) {
        if ((int)(ccount & 1) != group) continue;
        float ss = 0.f;   // sum of squares of this row's 128 columns of the chunk, before rounding
        const int db = (int)(ccount % Cfg::kDBufs);   // the group's accumulators alternate
        if (!dead && !mbar_wait(d_full_bar(db), (uint32_t)((ccount / Cfg::kDBufs) & 1))) timed_out();
        asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
#pragma unroll
        for (int g = 0; g < kChunkCols / 64; ++g) {
          const int64_t ecount = 2 * ccount + g;
          const int eslot = (int)(ecount % SE);
          uint32_t v[4][16];
#pragma unroll
          for (int i = 0; i < 4; ++i) tmem_ld16(lane_addr + (uint32_t)db * kChunkCols + g * 64 + i * 16, v[i]);
          asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
          if (g == kChunkCols / 64 - 1) {
            asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(d_empty_bar(db));
          }
          uint32_t slab;   // 32 rows x 128 B handed to the TMA store
          if (HAS_E) {
            if (!dead && !mbar_wait(e_full_bar(eslot, quarter), (uint32_t)((ecount / SE) & 1))) timed_out();
            slab = e_ring + (uint32_t)eslot * Cfg::kEStageBytes + (uint32_t)quarter * 4096;
          } else {
            // the store that last read this slab (two stores ago) must be done reading it
            if (lane == 0) bulk_wait_read<1>();
            __syncwarp();
            slab = slab0 + (uint32_t)g * 4096;
          }
          const uint32_t srow = slab + lane * 128;
          // all eight E pieces of the row first, so that their latencies overlap
          uint32_t e[8][4];
          if (HAS_E) {
#pragma unroll
            for (int c = 0; c < 8; ++c)
              asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];\n"
                           : "=r"(e[c][0]), "=r"(e[c][1]), "=r"(e[c][2]), "=r"(e[c][3])
                           : "r"(srow + ((c ^ (lane & 7)) << 4)));
          }
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            const uint32_t *w = &v[c >> 1][(c & 1) * 8];
            const uint32_t addr = srow + ((c ^ (lane & 7)) << 4);
            float f[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) f[i] = __uint_as_float(w[i]);
            if (HAS_E) {   // the sum replaces the E piece
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                f[2 * i] += __uint_as_float(e[c][i] << 16);
                f[2 * i + 1] += __uint_as_float(e[c][i] & 0xFFFF0000u);
              }
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) ss = fmaf(f[i], f[i], ss);
            const uint32_t o0 = pack_bf16(f[0], f[1]), o1 = pack_bf16(f[2], f[3]);
            const uint32_t o2 = pack_bf16(f[4], f[5]), o3 = pack_bf16(f[6], f[7]);
            asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};\n" ::"r"(addr), "r"(o0), "r"(o1), "r"(o2), "r"(o3)
                         : "memory");
          }
          asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
          __syncwarp();
          if (lane == 0) {
            if (rows_live) tma_store_3d_hint(&maps.out, slab, q * kChunkCols + g * 64, s1, s2, stream_out);
            bulk_commit();
            if (HAS_E) {
              // the store before this one is done reading its stage: hand that stage back; after
              // the chunk's last store wait for that one too, since this warp's next store is
              // two chunks away and the stage would sit idle until then
              if (g == kChunkCols / 64 - 1) {
                bulk_wait_read<0>();
                if (held >= 0) mbar_arrive(e_empty_bar(held, quarter));
                mbar_arrive(e_empty_bar(eslot, quarter));
              } else {
                bulk_wait_read<1>();
                if (held >= 0) mbar_arrive(e_empty_bar(held, quarter));
              }
            }
          }
          held = g == kChunkCols / 64 - 1 ? -1 : eslot;
        }
        if (a.rowsumsq != nullptr && tok < a.n) atomicAdd(a.rowsumsq + tok, ss);
      }
    }
    if (HAS_E && lane == 0) {
      bulk_wait_read<0>();
      if (held >= 0) mbar_arrive(e_empty_bar(held, quarter));
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
