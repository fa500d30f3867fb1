// d-split variant of the mma.sync codec kernel for calls with few rows per SM (the weight
// re-projection, small token batches).  A CTA takes one tile of 16*MT rows; its 8 warps share
// the rows and split the d index instead: in every 256-row stage of U, warp w owns 32-column
// chunk w.  Projection partials meet in shared memory, every warp then holds the full fp32
// coordinates and expands its own chunks.  Same fragment scheme and U layout as codec_mma.cuh.
#pragma once

#include "codec_mma.cuh"

namespace ssn {

constexpr int kDsplitStageRows = 256;   // 8 chunks of 32 columns: one per warp

template <int NT, int MT>
struct DsplitConfig {
  static constexpr int kRingBytes = kStages * UStageRing<NT, kDsplitStageRows>::kStageBytes;
  static constexpr int kRedBytes = kMmaWarps * MT * NT * 4 * 32 * 4;
  static constexpr int kSmemBytes = kRingBytes + kRedBytes;
};

template <int NT, int MT, bool SHIFT, int MODE>
__global__ void __launch_bounds__(kMmaThreads, 1) codec_mma_dsplit_kernel(const MmaArgs a) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  constexpr int KS = (NT + 1) / 2;
  constexpr bool has_project = (MODE & kModeProject) != 0;
  constexpr bool has_expand = (MODE & kModeExpand) != 0;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, tg = lane & 3;
  const int nchunks = a.d >> 5;
  const int nstage = (a.d + kDsplitStageRows - 1) / kDsplitStageRows;
  constexpr int kTileRows = 16 * MT;
  const int64_t ntiles = (a.n + kTileRows - 1) / kTileRows;
  const int64_t my_tiles = blockIdx.x < ntiles ? (ntiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;

  UStageRing<NT, kDsplitStageRows> ring;
  ring.U = a.U;
  ring.ldu = a.ldu;
  ring.d = a.d;
  ring.k = a.k;
  ring.nstage = nstage;
  ring.smem_base = smem_u32(smem_raw);
  ring.total_jobs = (int)my_tiles * ((has_project ? 1 : 0) + (has_expand ? 1 : 0)) * nstage;
  float *red = reinterpret_cast<float *>(smem_raw + DsplitConfig<NT, MT>::kRingBytes);
  int job = 0;
  ring.issue(0);
  ring.issue(1);
  const uint32_t lane_piece = (uint32_t)lane * 16;

  for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
    const int64_t tok0 = tile * kTileRows;
    const unsigned char *xrow[MT][2], *erow[MT][2], *prow[MT][2];
    int64_t tok[MT][2];
    bool own[MT][2];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int64_t t0 = tok0 + mt * 16 + h * 8 + g;
        own[mt][h] = t0 < a.n;
        const int64_t t = own[mt][h] ? t0 : a.n - 1;
        tok[mt][h] = t;
        xrow[mt][h] = has_project ? reinterpret_cast<const unsigned char *>(a.src + t * a.lds) + tg * 16 : nullptr;
        erow[mt][h] = g_zero_row + tg * 16;
        prow[mt][h] = g_zero_row + tg * 16;
        if (SHIFT && own[mt][h]) {
          // every warp looks the rows up; only warp 0 may raise the status bits
          ShiftTables quiet = a.shift;
          if (warp != 0) quiet.dev_status = nullptr;
          const int64_t er = embedding_row(quiet, t), pr = position_row(quiet, t);
          if (er >= 0)
            erow[mt][h] = reinterpret_cast<const unsigned char *>(
                              static_cast<const __nv_bfloat16 *>(a.shift.E) + er * a.shift.lde) + tg * 16;
          if (pr >= 0)
            prow[mt][h] = reinterpret_cast<const unsigned char *>(
                              static_cast<const __nv_bfloat16 *>(a.shift.P) + pr * a.shift.ldp) + tg * 16;
        }
      }

    float acc[MT][NT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[mt][nt][i] = 0.f;

    // ---------------------------------------------------------------- projection, my chunks
    if (has_project) {
      constexpr int NB = SHIFT ? 3 : 1;
      constexpr int kDepth = SHIFT ? 2 : 4;   // stages of row pieces in flight per warp
      uint4 buf[kDepth][MT][2][NB];
      auto load = [&](uint4 (&b)[MT][2][NB], int chunk) {
        const int off = min(chunk, nchunks - 1) * 64;
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            b[mt][h][0] = ldg16(xrow[mt][h] + off);
            if (SHIFT) {
              b[mt][h][1] = ldg16(erow[mt][h] + off);
              b[mt][h][2] = ldg16(prow[mt][h] + off);
            }
          }
      };
#pragma unroll
      for (int i = 0; i < kDepth; ++i) load(buf[i], i * 8 + warp);
      auto project_stage = [&](int st, uint4 (&b)[MT][2][NB]) {
        const uint32_t ubase = ring.acquire(job++);
        const int chunk = st * 8 + warp;
        uint32_t ra[MT][2][4];
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            if (SHIFT) {
              ra[mt][h][0] = sub3(b[mt][h][0].x, b[mt][h][1].x, b[mt][h][2].x);
              ra[mt][h][1] = sub3(b[mt][h][0].y, b[mt][h][1].y, b[mt][h][2].y);
              ra[mt][h][2] = sub3(b[mt][h][0].z, b[mt][h][1].z, b[mt][h][2].z);
              ra[mt][h][3] = sub3(b[mt][h][0].w, b[mt][h][1].w, b[mt][h][2].w);
            } else {
              ra[mt][h][0] = b[mt][h][0].x;
              ra[mt][h][1] = b[mt][h][0].y;
              ra[mt][h][2] = b[mt][h][0].z;
              ra[mt][h][3] = b[mt][h][0].w;
            }
          }
        load(b, chunk + 8 * kDepth);
        if (chunk < nchunks) {
          const uint32_t bbase = ubase + (uint32_t)warp * (NT * 512) + lane_piece;
          uint32_t bf[NT][4];
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) ldmatrix_x4_trans(bf[nt], bbase + nt * 512);
#pragma unroll
          for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
              mma_k16(acc[mt][nt], ra[mt][0][0], ra[mt][1][0], ra[mt][0][1], ra[mt][1][1], bf[nt][0], bf[nt][1]);
#pragma unroll
          for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
              mma_k16(acc[mt][nt], ra[mt][0][2], ra[mt][1][2], ra[mt][0][3], ra[mt][1][3], bf[nt][2], bf[nt][3]);
        }
      };
      for (int st = 0; st < nstage; st += kDepth) {
#pragma unroll
        for (int i = 0; i < kDepth; ++i)
          if (st + i < nstage) project_stage(st + i, buf[i]);
      }
      // partial sums of the 8 warps meet in shared memory; everybody leaves with the total
      __syncthreads();
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
          for (int i = 0; i < 4; ++i) red[((warp * MT + mt) * NT + nt) * 128 + i * 32 + lane] = acc[mt][nt][i];
      __syncthreads();
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            float s = 0.f;
#pragma unroll
            for (int w = 0; w < kMmaWarps; ++w) s += red[((w * MT + mt) * NT + nt) * 128 + i * 32 + lane];
            acc[mt][nt][i] = s;
          }
      __syncthreads();   // red is reused by the next tile

      if (a.zout != nullptr) {
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            if (!own[mt][h]) continue;
            __nv_bfloat16 *zrow = a.zout + tok[mt][h] * a.ldzout;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
              if ((nt & 7) != warp) continue;   // the column tiles are dealt to the warps
              const int col = nt * 8 + tg * 2;
              if (col < a.k) zrow[col] = __float2bfloat16_rn(acc[mt][nt][2 * h]);
              if (col + 1 < a.k) zrow[col + 1] = __float2bfloat16_rn(acc[mt][nt][2 * h + 1]);
            }
          }
      }
    }

    // ---------------------------------------------------------------- expansion, my chunks
    if (has_expand) {
      constexpr int parts = has_project ? 2 : 1;
      uint32_t za[parts][MT][KS][4];
      if (has_project) {
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
          for (int ks = 0; ks < KS; ++ks)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int nt = 2 * ks + (i >> 1), hh = i & 1;
              float v0 = 0.f, v1 = 0.f;
              if (nt < NT) {
                v0 = acc[mt][nt][2 * hh];
                v1 = acc[mt][nt][2 * hh + 1];
              }
              const uint32_t head = pack_bf16(v0, v1);
              za[0][mt][ks][i] = head;
              za[parts - 1][mt][ks][i] = pack_bf16(v0 - bf_lo(head), v1 - bf_hi(head));
            }
      } else {
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
          for (int ks = 0; ks < KS; ++ks)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int hh = i & 1, col = ks * 16 + (i >> 1) * 8 + tg * 2;
              uint32_t lo16 = 0, hi16 = 0;
              if (own[mt][hh]) {
                const unsigned short *zrow =
                    reinterpret_cast<const unsigned short *>(a.zin + tok[mt][hh] * a.ldzin);
                if (col < a.k) lo16 = zrow[col];
                if (col + 1 < a.k) hi16 = zrow[col + 1];
              }
              za[0][mt][ks][i] = lo16 | (hi16 << 16);
            }
      }
      unsigned char *orow[MT][2];
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int h = 0; h < 2; ++h)
          orow[mt][h] = reinterpret_cast<unsigned char *>(a.dst + tok[mt][h] * a.lddst) + tg * 16;

      constexpr int NBE = SHIFT ? 2 : 1;
      uint4 ebuf[2][MT][2][NBE];
      auto eload = [&](uint4 (&b)[MT][2][NBE], int chunk) {
        if (SHIFT) {
          const int off = min(chunk, nchunks - 1) * 64;
#pragma unroll
          for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              b[mt][h][0] = ldg16(erow[mt][h] + off);
              b[mt][h][1] = ldg16(prow[mt][h] + off);
            }
        }
      };
      eload(ebuf[0], warp);
      eload(ebuf[1], 8 + warp);
      const int rho = lane & 7, mi = lane >> 3;
      auto expand_stage = [&](int st, uint4 (&eb)[MT][2][NBE]) {
        const uint32_t ubase = ring.acquire(job++);
        const int chunk = st * 8 + warp;
        if (chunk < nchunks) {
          float o[MT][4][4];
#pragma unroll
          for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int j = 0; j < 4; ++j)
#pragma unroll
              for (int i = 0; i < 4; ++i) o[mt][j][i] = 0.f;
          const uint32_t blkbase = ubase + (uint32_t)warp * (NT * 512);
#pragma unroll
          for (int ks = 0; ks < KS; ++ks) {
            if (2 * ks + 1 < NT) {
#pragma unroll
              for (int jp = 0; jp < 2; ++jp) {
                uint32_t b[4];
                ldmatrix_x4(b, blkbase + (uint32_t)((((2 * ks + (mi & 1)) * 4) + 2 * jp + (mi >> 1)) * 8 + rho) * 16);
#pragma unroll
                for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                  for (int p = 0; p < parts; ++p) {
                    mma_k16(o[mt][2 * jp], za[p][mt][ks][0], za[p][mt][ks][1], za[p][mt][ks][2], za[p][mt][ks][3], b[0], b[1]);
                    mma_k16(o[mt][2 * jp + 1], za[p][mt][ks][0], za[p][mt][ks][1], za[p][mt][ks][2], za[p][mt][ks][3], b[2], b[3]);
                  }
              }
            } else {
              uint32_t b[4];
              ldmatrix_x4(b, blkbase + (uint32_t)((((NT - 1) * 4) + mi) * 8 + rho) * 16);
#pragma unroll
              for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int p = 0; p < parts; ++p)
#pragma unroll
                  for (int j = 0; j < 4; ++j) mma_k8(o[mt][j], za[p][mt][ks][0], za[p][mt][ks][1], b[j]);
            }
          }
          const int off = chunk * 64;
#pragma unroll
          for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              uint4 v;
              if (SHIFT) {
                v.x = add3(o[mt][0][2 * h], o[mt][0][2 * h + 1], eb[mt][h][0].x, eb[mt][h][1].x);
                v.y = add3(o[mt][1][2 * h], o[mt][1][2 * h + 1], eb[mt][h][0].y, eb[mt][h][1].y);
                v.z = add3(o[mt][2][2 * h], o[mt][2][2 * h + 1], eb[mt][h][0].z, eb[mt][h][1].z);
                v.w = add3(o[mt][3][2 * h], o[mt][3][2 * h + 1], eb[mt][h][0].w, eb[mt][h][1].w);
              } else {
                v.x = pack_bf16(o[mt][0][2 * h], o[mt][0][2 * h + 1]);
                v.y = pack_bf16(o[mt][1][2 * h], o[mt][1][2 * h + 1]);
                v.z = pack_bf16(o[mt][2][2 * h], o[mt][2][2 * h + 1]);
                v.w = pack_bf16(o[mt][3][2 * h], o[mt][3][2 * h + 1]);
              }
              if (own[mt][h]) *reinterpret_cast<uint4 *>(orow[mt][h] + off) = v;
            }
        }
        eload(eb, chunk + 16);
      };
      for (int st = 0; st < nstage; st += 2) {
        expand_stage(st, ebuf[0]);
        if (st + 1 < nstage) expand_stage(st + 1, ebuf[1]);
      }
    }
  }
  cp_async_wait<0>();
}

}  // namespace ssn
