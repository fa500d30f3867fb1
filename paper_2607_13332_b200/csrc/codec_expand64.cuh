// mma.sync expansion kernel with 64-column chunks and 256-bit global accesses (bf16, sm_100a):
//     Xhat = Z U^T + E[ids] + P[pos]          decompress
//
// The expansion is bound by the L1 / LSU front end (one "wavefront" per distinct row an
// instruction touches), not by DRAM: with 16-byte pieces every load and store instruction of a
// warp touches 8 rows.  This kernel halves that cost per byte by moving 32 bytes per thread per
// access (8 rows x 128 bytes per instruction: ld.global.nc.v8 / st.global.v8), and, when the
// positions are implicit (t mod seq_len) and the batch is a multiple of 16 sequences, it deals
// the tokens in tiles of 16 batch entries AT THE SAME POSITION, so the P piece of a tile is one
// broadcast load instead of 16 row loads.
//
// Fragment scheme: as in codec_mma.cuh, with the 64 columns of a chunk assigned to the MMA
// n-slots so that thread (g, tg) ends up with the 16 consecutive outputs at column 16*tg of rows
// g and g+8: output column of n-tile j, slot v is  16*(v/2) + 2*j + v%2.  U is staged in the
// matching fragment-major layout: piece (row dl, chunk c) at
//     (((dl/64)*NT + c)*8 + (dl/2)%8)*8 + ((dl/16)%4)*2 + dl%2      (16-byte units).
#pragma once

#include "codec_mma.cuh"

namespace ssn {

__device__ __forceinline__ void ldg32(const void *p, uint32_t (&r)[8]) {
  asm volatile("ld.global.nc.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "l"(p));
}
__device__ __forceinline__ void stg32(void *p, const uint32_t (&r)[8]) {
  asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};\n" ::"l"(p), "r"(r[0]), "r"(r[1]), "r"(r[2]),
               "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]) : "memory");
}

// U ring for 64-column chunks: 128 rows (two chunks) per stage.
template <int NT>
struct UStageRing64 {
  static constexpr int kStageBytes = kStageRows * NT * 16;
  const __nv_bfloat16 *U;
  int64_t ldu;
  int d, k, nstage, total_jobs;
  uint32_t smem_base;

  __device__ __forceinline__ void issue(int job) {
    if (job < total_jobs) {
      const int s = job % nstage;
      const int row0 = s * kStageRows;
      const int rows = min(kStageRows, d - row0);
      const uint32_t base = smem_base + (uint32_t)(job % kStages) * kStageBytes;
      for (int idx = threadIdx.x; idx < rows * NT; idx += kMmaThreads) {
        const int dl = idx / NT, c = idx - dl * NT;
        const int slot = (((dl >> 6) * NT + c) * 8 + ((dl >> 1) & 7)) * 8 + (((dl >> 4) & 3) << 1) + (dl & 1);
        const int valid = min(16, max(0, (k - 8 * c) * 2));
        cp_async16(base + slot * 16, U + (int64_t)(row0 + dl) * ldu + 8 * c, valid);
      }
    }
    cp_async_commit();
  }
  __device__ __forceinline__ uint32_t acquire(int job) {
    cp_async_wait<1>();
    __syncthreads();
    issue(job + 2);
    return smem_base + (uint32_t)(job % kStages) * kStageBytes;
  }
};

// NT = ceil(k/8) (rounded up by the launcher), MT = 16-token tiles per warp, SHIFT = add E and
// P, PDEDUP = tiles are 16 batch entries at one position (needs implicit positions).
template <int NT, int MT, bool SHIFT, bool PDEDUP>
__global__ void __launch_bounds__(kMmaThreads, 1) codec_expand64_kernel(const MmaArgs a) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  constexpr int KS = (NT + 1) / 2;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, tg = lane & 3;
  const int nchunks = a.d >> 6;

  UStageRing64<NT> ring;
  ring.U = a.U;
  ring.ldu = a.ldu;
  ring.d = a.d;
  ring.k = a.k;
  ring.nstage = (a.d + kStageRows - 1) / kStageRows;
  ring.smem_base = smem_u32(smem_raw);

  // tiles ("units") of 16 tokens, dealt to CTAs, rounds and warps
  const int64_t seq = a.shift.seq_len;
  const int64_t nbg = PDEDUP ? (a.n / seq) / 16 : 1;          // 16-sequence groups of the batch
  const int64_t nunits_all = PDEDUP ? seq * nbg : (a.n + 15) >> 4;
  const int64_t ulo = (nunits_all * blockIdx.x) / gridDim.x;
  const int64_t uhi = (nunits_all * (blockIdx.x + 1)) / gridDim.x;
  const int64_t ulen = uhi - ulo;
  constexpr int kRoundUnits = kMmaWarps * MT;
  const int rounds = (int)((ulen + kRoundUnits - 1) / kRoundUnits);
  ring.total_jobs = rounds * ring.nstage;
  int job = 0;
  ring.issue(0);
  ring.issue(1);

  for (int r = 0; r < rounds; ++r) {
    const int64_t rlo = ulo + (ulen * r) / rounds, rhi = ulo + (ulen * (r + 1)) / rounds;
    const int m = (int)(rhi - rlo), base = m / kMmaWarps, extra = m % kMmaWarps;
    const int nun = base + (warp < extra ? 1 : 0);
    const int64_t u0 = rlo + (int64_t)warp * base + min(warp, extra);

    const unsigned char *erow[MT][2], *prow[MT][2];
    unsigned char *orow[MT][2];
    int64_t tok[MT][2];
    bool own[MT][2];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int64_t u = u0 + mt;
        const int i = h * 8 + g;
        int64_t t;
        if (PDEDUP) {
          const int64_t p = u / nbg, bg = u - p * nbg;
          t = (bg * 16 + i) * seq + p;
          own[mt][h] = mt < nun;
        } else {
          t = u * 16 + i;
          own[mt][h] = mt < nun && t < a.n;
        }
        if (!own[mt][h]) t = 0;
        tok[mt][h] = t;
        orow[mt][h] = reinterpret_cast<unsigned char *>(a.dst + t * a.lddst) + tg * 32;
        erow[mt][h] = g_zero_row + tg * 32;
        prow[mt][h] = g_zero_row + tg * 32;
        if (SHIFT && own[mt][h]) {
          const int64_t er = embedding_row(a.shift, t), pr = position_row(a.shift, t);
          if (er >= 0)
            erow[mt][h] = reinterpret_cast<const unsigned char *>(
                              static_cast<const __nv_bfloat16 *>(a.shift.E) + er * a.shift.lde) + tg * 32;
          if (pr >= 0)
            prow[mt][h] = reinterpret_cast<const unsigned char *>(
                              static_cast<const __nv_bfloat16 *>(a.shift.P) + pr * a.shift.ldp) + tg * 32;
        }
      }

    // A fragments of the coordinates
    uint32_t za[MT][KS][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int ks = 0; ks < KS; ++ks)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int hh = i & 1, col = ks * 16 + (i >> 1) * 8 + tg * 2;
          uint32_t lo16 = 0, hi16 = 0;
          if (own[mt][hh]) {
            const unsigned short *zrow = reinterpret_cast<const unsigned short *>(a.zin + tok[mt][hh] * a.ldzin);
            if (col < a.k) lo16 = zrow[col];
            if (col + 1 < a.k) hi16 = zrow[col + 1];
          }
          za[mt][ks][i] = lo16 | (hi16 << 16);
        }

    // register ring (2 chunks) of the E pieces and of the P pieces (per row, or per tile)
    constexpr int PR = PDEDUP ? 1 : 2;
    uint32_t ebuf[2][MT][2][8], pbuf[2][MT][PR][8];
    auto eload = [&](uint32_t (&eb)[MT][2][8], uint32_t (&pb)[MT][PR][8], int chunk) {
      if (SHIFT) {
        const int off = min(chunk, nchunks - 1) * 128;
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
          for (int h = 0; h < 2; ++h) ldg32(erow[mt][h] + off, eb[mt][h]);
#pragma unroll
          for (int h = 0; h < PR; ++h) ldg32(prow[mt][h] + off, pb[mt][h]);
        }
      }
    };
    const int rho = lane & 7, mi = lane >> 3;
    auto expand_chunk = [&](uint32_t (&eb)[MT][2][8], uint32_t (&pb)[MT][PR][8], uint32_t ubase, int blk, int chunk) {
      float o[MT][8][4];
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int j = 0; j < 8; ++j)
#pragma unroll
          for (int i = 0; i < 4; ++i) o[mt][j][i] = 0.f;
      const uint32_t blkbase = ubase + (uint32_t)blk * (NT * 1024);
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        if (2 * ks + 1 < NT) {
#pragma unroll
          for (int jq = 0; jq < 4; ++jq) {
            uint32_t b[4];
            ldmatrix_x4(b, blkbase + (uint32_t)(((2 * ks + (mi & 1)) * 8 + 2 * jq + (mi >> 1)) * 8 + rho) * 16);
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
              mma_k16(o[mt][2 * jq], za[mt][ks][0], za[mt][ks][1], za[mt][ks][2], za[mt][ks][3], b[0], b[1]);
              mma_k16(o[mt][2 * jq + 1], za[mt][ks][0], za[mt][ks][1], za[mt][ks][2], za[mt][ks][3], b[2], b[3]);
            }
          }
        } else {
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            uint32_t b[4];
            ldmatrix_x4(b, blkbase + (uint32_t)(((NT - 1) * 8 + 4 * half + mi) * 8 + rho) * 16);
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
              for (int j = 0; j < 4; ++j) mma_k8(o[mt][4 * half + j], za[mt][ks][0], za[mt][ks][1], b[j]);
          }
        }
      }
      const int off = chunk * 128;
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          uint32_t v[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            if (SHIFT)
              v[j] = add3(o[mt][j][2 * h], o[mt][j][2 * h + 1], eb[mt][h][j], pb[mt][PDEDUP ? 0 : h][j]);
            else
              v[j] = pack_bf16(o[mt][j][2 * h], o[mt][j][2 * h + 1]);
          }
          if (own[mt][h]) stg32(orow[mt][h] + off, v);
        }
      eload(eb, pb, chunk + 2);
    };

    eload(ebuf[0], pbuf[0], 0);
    eload(ebuf[1], pbuf[1], 1);
    for (int c0 = 0; c0 < nchunks; c0 += 2) {
      const uint32_t ubase = ring.acquire(job++);
      expand_chunk(ebuf[0], pbuf[0], ubase, 0, c0);
      if (c0 + 1 < nchunks) expand_chunk(ebuf[1], pbuf[1], ubase, 1, c0 + 1);
    }
  }
  cp_async_wait<0>();
}

}  // namespace ssn
