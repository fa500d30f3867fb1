// Data-parallel device ops (include/agora_dp.h): the elementwise steps of an AsyncSPARTA round
// (Algorithm 3, Eq. sparta, Eq. delta_rule) and stage-wise gradient clipping (Sec. 4.3).  All of
// them stream their operands once: grid-stride loops, 128-bit accesses when every pointer is
// 16-byte aligned, a grid of two waves of resident blocks.
#include "agora_dp.h"

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdint>

namespace {

constexpr int kThreads = 256;
constexpr int kBlocksPerSm = 16;

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

int sm_count() {
  static int cached[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) n = 0;
    cached[dev] = n;
  }
  return cached[dev];
}

// blocks for `work` items handled one per thread and iteration
unsigned grid_for(int64_t work) {
  int64_t blocks = (work + kThreads - 1) / kThreads;
  const int64_t cap = (int64_t)(sm_count() > 0 ? sm_count() : 148) * kBlocksPerSm;
  if (blocks > cap) blocks = cap;
  return (unsigned)(blocks < 1 ? 1 : blocks);
}

ssn_status_t finish() { return cudaGetLastError() == cudaSuccess ? SSN_OK : SSN_ERR_CUDA; }

// ---- out[i] = f(a[i], b[i], c[i]) over floats, V = 4 (float4) or 1 ---------------------------
struct OpCopy {      // out = a
  __device__ float operator()(float a, float, float) const { return a; }
};
struct OpAxpy {      // out = c + w a      (c is the old value of out)
  float w;
  __device__ float operator()(float a, float, float c) const { return fmaf(w, a, c); }
};
struct OpApply {     // out = c + lambda (a - b)
  float lambda;
  __device__ float operator()(float a, float b, float c) const { return fmaf(lambda, a - b, c); }
};

template <int V, bool USE_B, bool USE_C, typename Op>
__global__ void __launch_bounds__(kThreads) ew_kernel(float *__restrict__ out, const float *__restrict__ a, const float *__restrict__ b, int64_t n, Op op) {
  const int64_t stride = (int64_t)gridDim.x * kThreads;
  if (V == 4) {
    const int64_t n4 = n >> 2;
    const float4 *a4 = reinterpret_cast<const float4 *>(a), *b4 = reinterpret_cast<const float4 *>(b);
    float4 *o4 = reinterpret_cast<float4 *>(out);
#pragma unroll 4
    for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < n4; i += stride) {
      const float4 x = a4[i];
      float4 y = make_float4(0.f, 0.f, 0.f, 0.f), z = y;
      if (USE_B) y = b4[i];
      if (USE_C) z = o4[i];
      o4[i] = make_float4(op(x.x, y.x, z.x), op(x.y, y.y, z.y), op(x.z, y.z, z.z), op(x.w, y.w, z.w));
    }
    // the last n % 4 elements
    const int64_t i = (n4 << 2) + (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (i < n) out[i] = op(a[i], USE_B ? b[i] : 0.f, USE_C ? out[i] : 0.f);
  } else {
#pragma unroll 4
    for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < n; i += stride)
      out[i] = op(a[i], USE_B ? b[i] : 0.f, USE_C ? out[i] : 0.f);
  }
}

template <bool USE_B, bool USE_C, typename Op>
ssn_status_t launch_ew(float *out, const float *a, const float *b, int64_t n, Op op, cudaStream_t s) {
  if (n == 0) return SSN_OK;
  const bool vec = aligned16(out) && aligned16(a) && (!USE_B || aligned16(b)) && n >= 4;
  if (vec)
    ew_kernel<4, USE_B, USE_C, Op><<<grid_for(n >> 2), kThreads, 0, s>>>(out, a, b, n, op);
  else
    ew_kernel<1, USE_B, USE_C, Op><<<grid_for(n), kThreads, 0, s>>>(out, a, b, n, op);
  return finish();
}

// ---- reducer: mean = acc / sum_w, deltas[i] = mean - chunks[i] -------------------------------
struct DeltaArgs {
  float *acc;
  const float *chunks[SPARTA_MAX_SENDERS];
  float *deltas[SPARTA_MAX_SENDERS];
  int64_t n;
  float inv_sum_w;
  int32_t senders;
};

template <int V>
__global__ void __launch_bounds__(kThreads) deltas_kernel(const DeltaArgs a) {
  const int64_t stride = (int64_t)gridDim.x * kThreads;
  if (V == 4) {
    const int64_t n4 = a.n >> 2;
    float4 *acc4 = reinterpret_cast<float4 *>(a.acc);
    for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < n4; i += stride) {
      float4 m = acc4[i];
      m.x *= a.inv_sum_w; m.y *= a.inv_sum_w; m.z *= a.inv_sum_w; m.w *= a.inv_sum_w;
      acc4[i] = m;
      for (int s = 0; s < a.senders; ++s) {
        const float4 c = reinterpret_cast<const float4 *>(a.chunks[s])[i];
        reinterpret_cast<float4 *>(a.deltas[s])[i] = make_float4(m.x - c.x, m.y - c.y, m.z - c.z, m.w - c.w);
      }
    }
    const int64_t i = (n4 << 2) + (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (i < a.n) {
      const float m = a.acc[i] * a.inv_sum_w;
      a.acc[i] = m;
      for (int s = 0; s < a.senders; ++s) a.deltas[s][i] = m - a.chunks[s][i];
    }
  } else {
    for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < a.n; i += stride) {
      const float m = a.acc[i] * a.inv_sum_w;
      a.acc[i] = m;
      for (int s = 0; s < a.senders; ++s) a.deltas[s][i] = m - a.chunks[s][i];
    }
  }
}

// ---- stage-wise clipping -------------------------------------------------------------------
template <typename T> __device__ __forceinline__ float widen(T v);
template <> __device__ __forceinline__ float widen<float>(float v) { return v; }
template <> __device__ __forceinline__ float widen<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T narrow(float v);
template <> __device__ __forceinline__ float narrow<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 narrow<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// 16 bytes of T per access when VEC
template <typename T, bool VEC>
__global__ void __launch_bounds__(kThreads) sumsq_kernel(const T *g, int64_t n, double *sumsq) {
  constexpr int E = VEC ? 16 / (int)sizeof(T) : 1;
  const int64_t stride = (int64_t)gridDim.x * kThreads;
  double acc = 0.0;
  if (VEC) {
    const int64_t nv = n / E;
    const uint4 *gv = reinterpret_cast<const uint4 *>(g);
    for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < nv; i += stride) {
      const uint4 raw = gv[i];
      const T *e = reinterpret_cast<const T *>(&raw);
      float part = 0.f;   // a handful of squares in fp32, then into the fp64 sum
#pragma unroll
      for (int j = 0; j < E; ++j) {
        const float v = widen<T>(e[j]);
        part = fmaf(v, v, part);
      }
      acc += (double)part;
    }
    const int64_t i = nv * E + (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (i < n) {
      const float v = widen<T>(g[i]);
      acc += (double)v * (double)v;
    }
  } else {
    for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < n; i += stride) {
      const float v = widen<T>(g[i]);
      acc += (double)v * (double)v;
    }
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
  __shared__ double warp_sums[kThreads / 32];
  if ((threadIdx.x & 31) == 0) warp_sums[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double total = 0.0;
    for (int w = 0; w < kThreads / 32; ++w) total += warp_sums[w];
    atomicAdd(sumsq, total);
  }
}

template <typename T, bool VEC>
__global__ void __launch_bounds__(kThreads) clip_scale_kernel(T *g, int64_t n, const double *sumsq, float threshold) {
  const float norm = (float)sqrt(*sumsq);
  const float coef = fminf(1.f, threshold / (norm + 1e-6f));
  if (!(coef < 1.f)) return;   // inside the budget: nothing to write
  constexpr int E = VEC ? 16 / (int)sizeof(T) : 1;
  const int64_t stride = (int64_t)gridDim.x * kThreads;
  if (VEC) {
    const int64_t nv = n / E;
    uint4 *gv = reinterpret_cast<uint4 *>(g);
    for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < nv; i += stride) {
      uint4 raw = gv[i];
      T *e = reinterpret_cast<T *>(&raw);
#pragma unroll
      for (int j = 0; j < E; ++j) e[j] = narrow<T>(widen<T>(e[j]) * coef);
      gv[i] = raw;
    }
    const int64_t i = nv * E + (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (i < n) g[i] = narrow<T>(widen<T>(g[i]) * coef);
  } else {
    for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < n; i += stride)
      g[i] = narrow<T>(widen<T>(g[i]) * coef);
  }
}

}  // namespace

extern "C" {

ssn_status_t sparta_segment(int64_t n_params, int32_t rounds_per_cycle, int64_t round, int64_t *lo,
                            int64_t *hi) {
  if (lo == nullptr || hi == nullptr) return SSN_ERR_NULL;
  if (n_params < 0 || rounds_per_cycle < 1 || round < 0 || n_params > (INT64_MAX / rounds_per_cycle))
    return SSN_ERR_SHAPE;
  const int64_t r = round % rounds_per_cycle;
  const int64_t a = n_params * r / rounds_per_cycle, b = n_params * (r + 1) / rounds_per_cycle;
  *lo = a & ~(int64_t)(SPARTA_SEGMENT_ALIGN - 1);
  *hi = r + 1 == rounds_per_cycle ? n_params : (b & ~(int64_t)(SPARTA_SEGMENT_ALIGN - 1));
  return SSN_OK;
}

ssn_status_t sparta_snapshot(const float *buf, int64_t lo, int64_t hi, float *snap, void *stream) {
  if (lo < 0 || hi < lo) return SSN_ERR_SHAPE;
  if (hi == lo) return SSN_OK;
  if (buf == nullptr || snap == nullptr) return SSN_ERR_NULL;
  return launch_ew<false, false>(snap, buf + lo, nullptr, hi - lo, OpCopy{}, static_cast<cudaStream_t>(stream));
}

ssn_status_t sparta_accumulate(float *acc, const float *chunk, float w, int64_t count, void *stream) {
  if (count < 0) return SSN_ERR_SHAPE;
  if (count == 0) return SSN_OK;
  if (acc == nullptr || chunk == nullptr) return SSN_ERR_NULL;
  return launch_ew<false, true>(acc, chunk, nullptr, count, OpAxpy{w}, static_cast<cudaStream_t>(stream));
}

ssn_status_t sparta_deltas(float *acc, float sum_w, const float *const *chunks, float *const *deltas,
                           int32_t senders, int64_t count, void *stream) {
  if (count < 0 || senders < 1 || senders > SPARTA_MAX_SENDERS || !(sum_w > 0.f)) return SSN_ERR_SHAPE;
  if (chunks == nullptr || deltas == nullptr) return SSN_ERR_NULL;
  if (count == 0) return SSN_OK;
  if (acc == nullptr) return SSN_ERR_NULL;
  DeltaArgs a{};
  a.acc = acc;
  a.n = count;
  a.inv_sum_w = 1.0f / sum_w;
  a.senders = senders;
  bool vec = aligned16(acc) && count >= 4;
  for (int32_t i = 0; i < senders; ++i) {
    if (chunks[i] == nullptr || deltas[i] == nullptr) return SSN_ERR_NULL;
    a.chunks[i] = chunks[i];
    a.deltas[i] = deltas[i];
    vec = vec && aligned16(chunks[i]) && aligned16(deltas[i]);
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (vec)
    deltas_kernel<4><<<grid_for(count >> 2), kThreads, 0, s>>>(a);
  else
    deltas_kernel<1><<<grid_for(count), kThreads, 0, s>>>(a);
  return finish();
}

ssn_status_t sparta_add_delta(float *buf, int64_t lo, int64_t hi, const float *delta, void *stream) {
  if (lo < 0 || hi < lo) return SSN_ERR_SHAPE;
  if (hi == lo) return SSN_OK;
  if (buf == nullptr || delta == nullptr) return SSN_ERR_NULL;
  return launch_ew<false, true>(buf + lo, delta, nullptr, hi - lo, OpAxpy{1.0f}, static_cast<cudaStream_t>(stream));
}

ssn_status_t sparta_apply_round(float *theta, int64_t lo, int64_t hi, const float *avg, const float *snap,
                                float lambda, void *stream) {
  if (lo < 0 || hi < lo) return SSN_ERR_SHAPE;
  if (hi == lo) return SSN_OK;
  if (theta == nullptr || avg == nullptr || snap == nullptr) return SSN_ERR_NULL;
  return launch_ew<true, true>(theta + lo, avg, snap, hi - lo, OpApply{lambda}, static_cast<cudaStream_t>(stream));
}

float stage_clip_threshold(int32_t n_stages, int32_t is_tail) {
  if (n_stages < 1) return 0.f;
  const float t = (float)(1.0 / std::sqrt((double)n_stages));
  return is_tail ? 2.f * t : t;
}

ssn_status_t stage_clip_sumsq(const void *grad, int64_t count, int32_t dtype, double *sumsq, void *stream) {
  if (dtype != SSN_F32 && dtype != SSN_BF16) return SSN_ERR_DTYPE;
  if (count < 0) return SSN_ERR_SHAPE;
  if (sumsq == nullptr) return SSN_ERR_NULL;
  if (count == 0) return SSN_OK;
  if (grad == nullptr) return SSN_ERR_NULL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const bool vec = aligned16(grad);
  if (dtype == SSN_F32) {
    const float *g = static_cast<const float *>(grad);
    if (vec) sumsq_kernel<float, true><<<grid_for(count / 4 + 1), kThreads, 0, s>>>(g, count, sumsq);
    else sumsq_kernel<float, false><<<grid_for(count), kThreads, 0, s>>>(g, count, sumsq);
  } else {
    const __nv_bfloat16 *g = static_cast<const __nv_bfloat16 *>(grad);
    if (vec) sumsq_kernel<__nv_bfloat16, true><<<grid_for(count / 8 + 1), kThreads, 0, s>>>(g, count, sumsq);
    else sumsq_kernel<__nv_bfloat16, false><<<grid_for(count), kThreads, 0, s>>>(g, count, sumsq);
  }
  return finish();
}

ssn_status_t stage_clip_scale(void *grad, int64_t count, int32_t dtype, const double *sumsq, float threshold,
                              void *stream) {
  if (dtype != SSN_F32 && dtype != SSN_BF16) return SSN_ERR_DTYPE;
  if (count < 0 || !(threshold > 0.f)) return SSN_ERR_SHAPE;
  if (sumsq == nullptr) return SSN_ERR_NULL;
  if (count == 0) return SSN_OK;
  if (grad == nullptr) return SSN_ERR_NULL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const bool vec = aligned16(grad);
  if (dtype == SSN_F32) {
    float *g = static_cast<float *>(grad);
    if (vec) clip_scale_kernel<float, true><<<grid_for(count / 4 + 1), kThreads, 0, s>>>(g, count, sumsq, threshold);
    else clip_scale_kernel<float, false><<<grid_for(count), kThreads, 0, s>>>(g, count, sumsq, threshold);
  } else {
    __nv_bfloat16 *g = static_cast<__nv_bfloat16 *>(grad);
    if (vec) clip_scale_kernel<__nv_bfloat16, true><<<grid_for(count / 8 + 1), kThreads, 0, s>>>(g, count, sumsq, threshold);
    else clip_scale_kernel<__nv_bfloat16, false><<<grid_for(count), kThreads, 0, s>>>(g, count, sumsq, threshold);
  }
  return finish();
}

}  // extern "C"
