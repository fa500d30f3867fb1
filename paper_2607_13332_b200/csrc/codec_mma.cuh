// Tensor-core kernels of the SSN codec for bf16 (sm_100a).
//
// One kernel template covers the three shapes the codec needs:
//   project          Z = (X - E[ids] - P[pos]) U              compress, grad-project (coeff)
//   expand           Xhat = Z U^T + E[ids] + P[pos]           decompress
//   project+expand   Y = (X U) U^T, coordinates kept in fp32  grad-project (full), re-projection
//
// Data flow.  The big operands (X, gathered E rows, P rows, the output) never touch shared
// memory: every thread moves 16-byte pieces (8 bf16) of its own rows between global memory and
// registers, forms the residual in fp32 and feeds it to mma.sync.m16n8k16 as the A operand.
// A contraction does not care in which order the contracted index is visited, so the 32
// columns of a chunk are assigned to MMA k-slots in the order that makes each thread's natural
// 16-byte piece its own A fragment; U is laid out in shared memory to match ("fragment-major":
// the eight 16-byte rows of every 8x8 ldmatrix tile are contiguous, hence conflict-free).  U is
// streamed through a 3-stage cp.async ring, 128 rows of d per stage, shared by the 8 warps.
//
// Work split.  The grid is sized to the machine; CTA b owns the contiguous token range
// [n*b/G, n*(b+1)/G) and walks it in equal rounds, each round giving every warp the same
// number (<= 16*MT) of tokens.  All CTAs therefore finish together; rows a warp does not own
// are computed on clamped addresses and never stored.
#pragma once

#include "codec_mma_launch.h"
#include "ssn_common.cuh"

namespace ssn {

constexpr int kMmaWarps = 8;
constexpr int kMmaThreads = kMmaWarps * 32;
constexpr int kStageRows = 128;   // rows of U (values of the d index) per pipeline stage
constexpr int kStages = 3;
constexpr int kZeroRowBytes = 65536;

// A row of zeros that stands in for the E / P row of a token that has none (absent table,
// index out of range, row past the end of the batch).  Never written.  One copy per translation
// unit that gathers rows.
static __device__ __align__(128) unsigned char g_zero_row[kZeroRowBytes];


// ---- small PTX wrappers --------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, int src_bytes) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes));
}
// the same, not allocating in L1 (for rows that are read once)
__device__ __forceinline__ void cp_async16_cg(uint32_t dst, const void *src) {
  asm volatile("cp.async.cg.shared.global.L2::256B [%0], [%1], 16;\n" ::"r"(dst), "l"(src));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_k16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                        uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
      "{%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_k8(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t b0) {
  asm volatile(
      "mma.sync.aligned.m16n8k8.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, "
      "{%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(b0));
}
__device__ __forceinline__ uint4 ldg16(const void *p) {
  return __ldg(reinterpret_cast<const uint4 *>(p));
}
__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}
// Packed pair of fp32 in one 64-bit register (sm_100a has two-wide fp32 add/sub).
__device__ __forceinline__ unsigned long long f32x2_of(uint32_t w) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(w << 16), "r"(w & 0xffff0000u));
  return r;
}
__device__ __forceinline__ unsigned long long f32x2_make(float lo, float hi) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ uint32_t f32x2_to_bf16x2(unsigned long long v) {
  uint32_t lo, hi, o;
  asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(v));
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(o) : "r"(hi), "r"(lo));
  return o;
}
// (x - e) - p on a pair of packed bf16, in fp32, rounded once to bf16.
__device__ __forceinline__ uint32_t sub3(uint32_t x, uint32_t e, uint32_t p) {
  unsigned long long r;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(f32x2_of(x)), "l"(f32x2_of(e)));
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(r), "l"(f32x2_of(p)));
  return f32x2_to_bf16x2(r);
}
// (acc + e) + p, rounded once.
__device__ __forceinline__ uint32_t add3(float a0, float a1, uint32_t e, uint32_t p) {
  unsigned long long r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(f32x2_make(a0, a1)), "l"(f32x2_of(e)));
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(r), "l"(f32x2_of(p)));
  return f32x2_to_bf16x2(r);
}

// ---- the U stage ring ------------------------------------------------------------------------
// Piece (row dl of the stage, 16-byte column chunk c) goes to slot
//   (((dl/32)*NT + c)*4 + ((dl/2)%4))*8 + ((dl/8)%4)*2 + dl%2
// so that the four 8x8 tiles a warp fetches for one (32-row block, chunk) are 512 contiguous
// bytes, both for the transposed loads of the projection and the plain loads of the expansion.
template <int NT, int ROWS = kStageRows>
struct UStageRing {
  static constexpr int kStageBytes = ROWS * NT * 16;
  const __nv_bfloat16 *U;
  int64_t ldu;
  int d, k, nstage, total_jobs;
  uint32_t smem_base;
  bool named_barrier = false;   // the kMmaThreads users are only part of the CTA

  __device__ __forceinline__ void issue(int job) {
    if (job < total_jobs) {
      const int s = job % nstage;
      const int row0 = s * ROWS;
      const int rows = min(ROWS, d - row0);
      const uint32_t base = smem_base + (uint32_t)(job % kStages) * kStageBytes;
      for (int idx = threadIdx.x; idx < rows * NT; idx += kMmaThreads) {
        const int dl = idx / NT, c = idx - dl * NT;
        const int slot = (((dl >> 5) * NT + c) * 4 + ((dl >> 1) & 3)) * 8 + (((dl >> 3) & 3) << 1) + (dl & 1);
        const int valid = min(16, max(0, (k - 8 * c) * 2));
        cp_async16(base + slot * 16, U + (int64_t)(row0 + dl) * ldu + 8 * c, valid);
      }
    }
    cp_async_commit();
  }
  // Makes stage `job` readable by every warp and refills the buffer freed by job-1.
  __device__ __forceinline__ uint32_t acquire(int job) {
    cp_async_wait<1>();
    if (named_barrier)
      asm volatile("bar.sync 1, %0;\n" ::"n"(kMmaThreads) : "memory");
    else
      __syncthreads();
    issue(job + 2);
    return smem_base + (uint32_t)(job % kStages) * kStageBytes;
  }
};

// ---- the kernel --------------------------------------------------------------------------------
// NT >= ceil(k / 8) column tiles of U; MT = 16-row token tiles per warp; SHIFT = the E/P terms
// take part (subtracted while projecting, added while expanding); MODE = which passes run.
constexpr int kModeProject = 1, kModeExpand = 2, kModeBoth = 3;

template <int NT, int MT, bool SHIFT, int MODE>
__global__ void __launch_bounds__(kMmaThreads, 1) codec_mma_kernel(const MmaArgs a) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  constexpr int KS = (NT + 1) / 2;   // k-steps of 16 coordinates (the last may be half)
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, tg = lane & 3;
  constexpr bool has_project = (MODE & kModeProject) != 0;
  constexpr bool has_expand = (MODE & kModeExpand) != 0;
  const int nchunks = a.d >> 5;

  UStageRing<NT> ring;
  ring.U = a.U;
  ring.ldu = a.ldu;
  ring.d = a.d;
  ring.k = a.k;
  ring.nstage = (a.d + kStageRows - 1) / kStageRows;
  ring.smem_base = smem_u32(smem_raw);

  const int64_t lo = (a.n * blockIdx.x) / gridDim.x;
  const int64_t hi = (a.n * (blockIdx.x + 1)) / gridDim.x;
  const int64_t len = hi - lo;
  constexpr int kRound = kMmaWarps * 16 * MT;
  const int rounds = (int)((len + kRound - 1) / kRound);
  ring.total_jobs = rounds * ((has_project ? 1 : 0) + (has_expand ? 1 : 0)) * ring.nstage;
  int job = 0;
  ring.issue(0);
  ring.issue(1);

  const uint32_t lane_piece = (uint32_t)lane * 16;   // ldmatrix: lane l supplies row l%8 of tile l/8

  for (int r = 0; r < rounds; ++r) {
    const int64_t rlo = lo + (len * r) / rounds, rhi = lo + (len * (r + 1)) / rounds;
    const int per_warp = (int)((rhi - rlo + kMmaWarps - 1) / kMmaWarps);
    const int64_t wlo = rlo + (int64_t)warp * per_warp;
    const int wcount = (int)max((int64_t)0, min((int64_t)per_warp, rhi - wlo));

    // per-thread rows: (mt, h) -> token wlo + mt*16 + h*8 + g
    const unsigned char *xrow[MT][2], *erow[MT][2], *prow[MT][2];
    int64_t tok[MT][2];
    bool own[MT][2];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int ri = mt * 16 + h * 8 + g;
        own[mt][h] = ri < wcount;
        const int64_t t = own[mt][h] ? wlo + ri : min(wlo, a.n - 1);
        tok[mt][h] = t;
        xrow[mt][h] = has_project ? reinterpret_cast<const unsigned char *>(a.src + t * a.lds) + tg * 16 : nullptr;
        erow[mt][h] = g_zero_row + tg * 16;
        prow[mt][h] = g_zero_row + tg * 16;
        if (SHIFT && own[mt][h]) {
          const int64_t er = embedding_row(a.shift, t), pr = position_row(a.shift, t);
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

    // ------------------------------------------------------------------ projection pass
    if (has_project) {
      // A ring of register buffers, one 32-column chunk each.  A buffer is refilled (chunk
      // c + kPBuf) as soon as its contents have been turned into A fragments, before the MMAs
      // of chunk c are issued, so close to kPBuf chunks of loads are in flight per thread.
      constexpr int NB = SHIFT ? 3 : 1;
      constexpr int kPBuf = SHIFT ? 2 : 4;
      uint4 buf[kPBuf][MT][2][NB];
      auto load = [&](uint4 (&b)[MT][2][NB], int off) {
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
      auto convert = [&](uint4 (&b)[MT][2][NB], uint32_t (&ra)[MT][2][4]) {
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
      };
      auto mmas = [&](uint32_t (&ra)[MT][2][4], uint32_t ubase, int blk) {
        const uint32_t bbase = ubase + (uint32_t)blk * (NT * 512) + lane_piece;
        uint32_t b[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) ldmatrix_x4_trans(b[nt], bbase + nt * 512);
        // the two MMAs that share an accumulator are issued NT*MT instructions apart
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
          for (int mt = 0; mt < MT; ++mt)
            mma_k16(acc[mt][nt], ra[mt][0][0], ra[mt][1][0], ra[mt][0][1], ra[mt][1][1], b[nt][0], b[nt][1]);
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
          for (int mt = 0; mt < MT; ++mt)
            mma_k16(acc[mt][nt], ra[mt][0][2], ra[mt][1][2], ra[mt][0][3], ra[mt][1][3], b[nt][2], b[nt][3]);
      };

#pragma unroll
      for (int i = 0; i < kPBuf; ++i)
        if (i < nchunks) load(buf[i], i * 64);
      for (int c0 = 0; c0 < nchunks; c0 += 4) {
        const uint32_t ubase = ring.acquire(job++);
        const int base_off = c0 * 64;
#pragma unroll
        for (int cc = 0; cc < 4; ++cc) {
          if (c0 + cc < nchunks) {
            uint32_t ra[MT][2][4];
            convert(buf[cc % kPBuf], ra);
            if (c0 + cc + kPBuf < nchunks) load(buf[cc % kPBuf], base_off + (cc + kPBuf) * 64);
            mmas(ra, ubase, cc);
          }
        }
      }

      if (a.zout != nullptr) {
        const bool vec = ((a.ldzout & 1) == 0) && ((reinterpret_cast<uintptr_t>(a.zout) & 3) == 0);
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            if (!own[mt][h]) continue;
            __nv_bfloat16 *zrow = a.zout + tok[mt][h] * a.ldzout;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
              const int col = nt * 8 + tg * 2;
              const float v0 = acc[mt][nt][2 * h], v1 = acc[mt][nt][2 * h + 1];
              if (vec && col + 1 < a.k) {
                *reinterpret_cast<uint32_t *>(zrow + col) = pack_bf16(v0, v1);
              } else {
                if (col < a.k) zrow[col] = __float2bfloat16_rn(v0);
                if (col + 1 < a.k) zrow[col + 1] = __float2bfloat16_rn(v1);
              }
            }
          }
      }
    }

    // ------------------------------------------------------------------ expansion pass
    if (has_expand) {
      // A fragments of the coordinates: exact bf16 when read from memory, split into a bf16
      // head and a bf16 remainder (two MMAs) when they come from the fp32 accumulators.
      constexpr int parts = has_project ? 2 : 1;
      uint32_t za[parts][MT][KS][4];
      if (has_project) {
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
          for (int ks = 0; ks < KS; ++ks)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              // i: 0 -> (row g, tile 2ks), 1 -> (row g+8, tile 2ks), 2/3 -> tile 2ks+1
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

      // Register ring of kEBuf chunks of E/P pieces: the buffer of chunk c is refilled with
      // chunk c + kEBuf right after it has been added to the accumulators.
      constexpr int NBE = SHIFT ? 2 : 1;
      constexpr int kEBuf = 4;
      uint4 ebuf[kEBuf][MT][2][NBE];
      auto eload = [&](uint4 (&buf)[MT][2][NBE], int off) {
        if (SHIFT) {
#pragma unroll
          for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              buf[mt][h][0] = ldg16(erow[mt][h] + off);
              buf[mt][h][1] = ldg16(prow[mt][h] + off);
            }
        }
      };
      auto ecompute = [&](uint4 (&buf)[MT][2][NBE], uint32_t ubase, int blk, int off, bool refill) {
        float o[MT][4][4];
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
          for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int i = 0; i < 4; ++i) o[mt][j][i] = 0.f;
        const uint32_t blkbase = ubase + (uint32_t)blk * (NT * 512);
        const int rho = lane & 7, mi = lane >> 3;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
          if (2 * ks + 1 < NT) {
            // full k-step: tiles (j, j+1) x chunks (2ks, 2ks+1) per ldmatrix.x4
#pragma unroll
            for (int jp = 0; jp < 2; ++jp) {
              uint32_t b[4];
              const uint32_t addr = blkbase + (uint32_t)((((2 * ks + (mi & 1)) * 4) + 2 * jp + (mi >> 1)) * 8 + rho) * 16;
              ldmatrix_x4(b, addr);
#pragma unroll
              for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int p = 0; p < parts; ++p) {
                  mma_k16(o[mt][2 * jp], za[p][mt][ks][0], za[p][mt][ks][1], za[p][mt][ks][2],
                          za[p][mt][ks][3], b[0], b[1]);
                  mma_k16(o[mt][2 * jp + 1], za[p][mt][ks][0], za[p][mt][ks][1], za[p][mt][ks][2],
                          za[p][mt][ks][3], b[2], b[3]);
                }
            }
          } else {
            // half k-step (NT odd): chunk NT-1 of the four tiles in one ldmatrix.x4
            uint32_t b[4];
            const uint32_t addr = blkbase + (uint32_t)((((NT - 1) * 4) + mi) * 8 + rho) * 16;
            ldmatrix_x4(b, addr);
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
              for (int p = 0; p < parts; ++p)
#pragma unroll
                for (int j = 0; j < 4; ++j) mma_k8(o[mt][j], za[p][mt][ks][0], za[p][mt][ks][1], b[j]);
          }
        }
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            uint4 v;
            if (SHIFT) {
              v.x = add3(o[mt][0][2 * h], o[mt][0][2 * h + 1], buf[mt][h][0].x, buf[mt][h][1].x);
              v.y = add3(o[mt][1][2 * h], o[mt][1][2 * h + 1], buf[mt][h][0].y, buf[mt][h][1].y);
              v.z = add3(o[mt][2][2 * h], o[mt][2][2 * h + 1], buf[mt][h][0].z, buf[mt][h][1].z);
              v.w = add3(o[mt][3][2 * h], o[mt][3][2 * h + 1], buf[mt][h][0].w, buf[mt][h][1].w);
            } else {
              v.x = pack_bf16(o[mt][0][2 * h], o[mt][0][2 * h + 1]);
              v.y = pack_bf16(o[mt][1][2 * h], o[mt][1][2 * h + 1]);
              v.z = pack_bf16(o[mt][2][2 * h], o[mt][2][2 * h + 1]);
              v.w = pack_bf16(o[mt][3][2 * h], o[mt][3][2 * h + 1]);
            }
            if (own[mt][h]) *reinterpret_cast<uint4 *>(orow[mt][h] + off) = v;
          }
        if (refill) eload(buf, off + kEBuf * 64);
      };

#pragma unroll
      for (int i = 0; i < kEBuf; ++i)
        if (i < nchunks) eload(ebuf[i], i * 64);
      for (int c0 = 0; c0 < nchunks; c0 += 4) {
        const uint32_t ubase = ring.acquire(job++);
        const int base_off = c0 * 64;
#pragma unroll
        for (int cc = 0; cc < 4; ++cc)
          if (c0 + cc < nchunks)
            ecompute(ebuf[cc % kEBuf], ubase, cc, base_off + cc * 64, c0 + cc + kEBuf < nchunks);
      }
    }
  }
  cp_async_wait<0>();
}

}  // namespace ssn
