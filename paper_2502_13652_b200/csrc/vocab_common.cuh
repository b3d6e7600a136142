// Helpers shared by the two vocabulary-pass kernels: 16-byte vector access for bf16 / fp32
// rows, the device-side row list, and the even partition of the active rows over the grid.
#pragma once

#include "c2t_internal.h"

namespace c2t {
namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr int kWarps = kPassThreads / 32;
constexpr unsigned kFull = 0xFFFFFFFFu;

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ uint4 ldg_stream(const uint4 *p) {
  uint4 v;
  asm("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

__device__ __forceinline__ uint32_t max_nan_bf16x2(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("max.NaN.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
__device__ __forceinline__ uint32_t max_bf16x2(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
__device__ __forceinline__ float max_nan_f32(float a, float b) {
  float d;
  asm("max.NaN.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
  return d;
}

// -inf is read as -2^127: finite, and still finite after a multiplication by log2(e)
constexpr uint32_t kLowestBf16x2 = 0xFF00FF00u;   // two copies of -2^127 in bf16
constexpr float kLowestF32 = -1.7014118346046923e38f;

template <bool BF16>
struct Vec {
  static constexpr int N = BF16 ? 8 : 4;

  // -inf -> lowest finite; NaN stays NaN
  __device__ static __forceinline__ void clamp(uint4 &q) {
    if (BF16) {
      q.x = max_nan_bf16x2(q.x, kLowestBf16x2);
      q.y = max_nan_bf16x2(q.y, kLowestBf16x2);
      q.z = max_nan_bf16x2(q.z, kLowestBf16x2);
      q.w = max_nan_bf16x2(q.w, kLowestBf16x2);
    } else {
      q.x = __float_as_uint(max_nan_f32(__uint_as_float(q.x), kLowestF32));
      q.y = __float_as_uint(max_nan_f32(__uint_as_float(q.y), kLowestF32));
      q.z = __float_as_uint(max_nan_f32(__uint_as_float(q.z), kLowestF32));
      q.w = __float_as_uint(max_nan_f32(__uint_as_float(q.w), kLowestF32));
    }
  }
  // maximum of the vector, NaNs ignored (NaN only if every element is NaN)
  __device__ static __forceinline__ float vmax(const uint4 &q) {
    if (BF16) {
      uint32_t m = max_bf16x2(max_bf16x2(q.x, q.y), max_bf16x2(q.z, q.w));
      return fmaxf(__uint_as_float(m << 16), __uint_as_float(m & 0xFFFF0000u));
    }
    return fmaxf(fmaxf(__uint_as_float(q.x), __uint_as_float(q.y)),
                 fmaxf(__uint_as_float(q.z), __uint_as_float(q.w)));
  }
  __device__ static __forceinline__ void unpack(const uint4 &q, float *x) {
    if (BF16) {
      x[0] = __uint_as_float(q.x << 16); x[1] = __uint_as_float(q.x & 0xFFFF0000u);
      x[2] = __uint_as_float(q.y << 16); x[3] = __uint_as_float(q.y & 0xFFFF0000u);
      x[4] = __uint_as_float(q.z << 16); x[5] = __uint_as_float(q.z & 0xFFFF0000u);
      x[6] = __uint_as_float(q.w << 16); x[7] = __uint_as_float(q.w & 0xFFFF0000u);
    } else {
      x[0] = __uint_as_float(q.x); x[1] = __uint_as_float(q.y);
      x[2] = __uint_as_float(q.z); x[3] = __uint_as_float(q.w);
    }
  }
  // vector v of a row; the last vector of a row whose length is not a multiple of N is
  // assembled from scalar loads and padded with the lowest finite value
  __device__ static __forceinline__ uint4 load(const void *row, int v, int v_full, int V) {
    if (v < v_full) return ldg_stream(reinterpret_cast<const uint4 *>(row) + v);
    uint4 q;
    if (BF16) {
      const uint16_t *e = reinterpret_cast<const uint16_t *>(row) + (size_t)v * 8;
      uint32_t w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        uint32_t lo = (v * 8 + 2 * i < V) ? e[2 * i] : 0xFF00u;
        uint32_t hi = (v * 8 + 2 * i + 1 < V) ? e[2 * i + 1] : 0xFF00u;
        w[i] = lo | (hi << 16);
      }
      q = make_uint4(w[0], w[1], w[2], w[3]);
    } else {
      const uint32_t *e = reinterpret_cast<const uint32_t *>(row) + (size_t)v * 4;
      const uint32_t low = __float_as_uint(kLowestF32);
      q.x = (v * 4 + 0 < V) ? e[0] : low;
      q.y = (v * 4 + 1 < V) ? e[1] : low;
      q.z = (v * 4 + 2 < V) ? e[2] : low;
      q.w = (v * 4 + 3 < V) ? e[3] : low;
    }
    return q;
  }
};

// Exclusive prefix sums of the clamped per-sequence row counts into s_off[0..B]; returns the total.
__device__ int build_row_offsets(const int32_t *counts, int B, int cap, int *s_off) {
  const int tid = threadIdx.x, lane = tid & 31;
  for (int i = tid; i < B; i += blockDim.x) {
    int c = counts[i];
    s_off[i + 1] = c < 0 ? 0 : (c > cap ? cap : c);
  }
  if (tid == 0) s_off[0] = 0;
  __syncthreads();
  if (tid < 32) {
    int carry = 0;
    for (int base = 1; base <= B; base += 32) {
      int i = base + lane;
      int v = i <= B ? s_off[i] : 0;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(kFull, v, o);
        if (lane >= o) v += t;
      }
      v += carry;
      if (i <= B) s_off[i] = v;
      carry = __shfl_sync(kFull, v, 31);
    }
  }
  __syncthreads();
  return s_off[B];
}

// largest b with s_off[b] <= a
__device__ __forceinline__ int find_sequence(const int *s_off, int B, int a) {
  int lo = 0, hi = B;
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (s_off[mid] <= a) lo = mid; else hi = mid;
  }
  return lo;
}

struct Partition {
  int n_rows, vec_per_row, v_full;
  long long span, start, end;
};

template <int VEC>
__device__ __forceinline__ Partition make_partition(const PassParams &p, int n_rows) {
  Partition pt;
  pt.n_rows = n_rows;
  pt.vec_per_row = (p.V + VEC - 1) / VEC;
  pt.v_full = p.V / VEC;
  long long W = (long long)n_rows * pt.vec_per_row;
  long long span = (W + gridDim.x - 1) / gridDim.x;
  pt.span = span < kMinSpanVectors ? kMinSpanVectors : span;
  pt.start = (long long)blockIdx.x * pt.span;
  pt.end = pt.start + pt.span < W ? pt.start + pt.span : W;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    p.info->n_rows = n_rows;
    p.info->vec_per_row = pt.vec_per_row;
    p.info->span = pt.span;
    p.info->pad = 0;
  }
  return pt;
}


}  // namespace
}  // namespace c2t
