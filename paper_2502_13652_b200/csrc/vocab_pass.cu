// The vocabulary pass: one streaming read of every active logits row.
//
// expand_pass_kernel  — per row: softmax normaliser and entropy sums plus the K largest
//                       logits (ties to the lower token id)      (Sec. 4.2.1, Eq. 2, Sec. 4.2.2)
// argmax_pass_kernel  — per row: the largest logit (ties to the lower token id), for the
//                       greedy acceptance walk                    (Sec. 5 Metrics)
//
// Work partition.  The active rows (a device-side count per sequence) are laid end to end as
// n_rows * vec_per_row 16-byte vectors and cut into equal contiguous spans, one per CTA of a
// persistent grid (2 CTAs per SM), so every CTA streams the same number of bytes whatever the
// row count.  A span may cover the tail of one row, some whole rows and the head of another;
// each (row, CTA) piece is a "segment" and produces one partial record.  The pruning kernel
// merges the partials of a row in double precision.
//
// Sums.  A segment accumulates, in fp32, S = sum e^(x - m) and T = sum e^(x - m) (x - m) over
// all its elements EXCEPT its own K largest, which leave the kernel as exact (value, token)
// keys and are added in double precision by the merge.  The dominant terms of a peaked row
// are therefore exact, and the fp32 sums only carry the tail.  m is a per-thread reference
// (any value within 60 of everything the thread adds), not necessarily the maximum.
//
// Top-K.  The CTA keeps a K-slot list in shared memory.  A new key is inserted by walking
// the slots with atomicMax, carrying the smaller key onwards; what falls off the end was
// evicted.  Every evicted key is smaller than all final entries, so the largest evicted key
// is an exact filter for later elements; its value part is the fast test applied to the
// maximum of each 16-byte vector.  A warm-up over the first vector of every thread seeds the
// filter with the K-th largest vector maximum.
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
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
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

constexpr uint32_t kLowestBf16x2 = 0xFF7FFF7Fu;   // two copies of the lowest finite bf16
constexpr float kLowestF32 = -3.4028234663852886e38f;

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
        uint32_t lo = (v * 8 + 2 * i < V) ? e[2 * i] : 0xFF7Fu;
        uint32_t hi = (v * 8 + 2 * i + 1 < V) ? e[2 * i + 1] : 0xFF7Fu;
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
  }
  return pt;
}

// ---------------------------------------------------------------- expand ----

struct Acc {
  float m, S0, S1, T0, T1;
};

__device__ __forceinline__ void acc_rescale(Acc &a, float new_m) {
  float d = fmaxf(a.m - new_m, -1e30f);
  float f = ex2f(d * kLog2e);
  float S = a.S0 + a.S1, T = a.T0 + a.T1;
  a.T0 = f * (T + d * S);
  a.T1 = 0.f;
  a.S0 = S * f;
  a.S1 = 0.f;
  a.m = new_m;
}

__device__ __forceinline__ void acc_scalar(Acc &a, float x) {
  if (x - a.m > 60.f) acc_rescale(a, x);
  float d = x - a.m;
  float e = ex2f(d * kLog2e);
  a.S0 += e;
  a.T0 = fmaf(e, d, a.T0);
}

template <bool BF16>
__device__ __forceinline__ void acc_vector(Acc &a, const uint4 &q) {
  float x[Vec<BF16>::N];
  Vec<BF16>::unpack(q, x);
#pragma unroll
  for (int i = 0; i < Vec<BF16>::N; i += 2) {
    float d0 = x[i] - a.m, d1 = x[i + 1] - a.m;
    float e0 = ex2f(d0 * kLog2e), e1 = ex2f(d1 * kLog2e);
    a.S0 += e0;
    a.S1 += e1;
    a.T0 = fmaf(e0, d0, a.T0);
    a.T1 = fmaf(e1, d1, a.T1);
  }
}

__device__ __forceinline__ void combine(float &m, float &S, float &T, float m2, float S2, float T2) {
  float M = fmaxf(m, m2);
  float d1 = fmaxf(m - M, -1e30f), d2 = fmaxf(m2 - M, -1e30f);
  float f1 = ex2f(d1 * kLog2e), f2 = ex2f(d2 * kLog2e);
  T = f1 * (T + d1 * S) + f2 * (T2 + d2 * S2);
  S = f1 * S + f2 * S2;
  m = M;
}

// Rare path: the vector holds at least one element not below the filter.
template <bool BF16>
__device__ __noinline__ void slow_vector(const uint4 &q, uint32_t tok0, int K, Acc &acc, float &thr,
                                         unsigned long long *s_list, unsigned long long *s_thrkey) {
  float x[Vec<BF16>::N];
  Vec<BF16>::unpack(q, x);
  unsigned long long tk = *reinterpret_cast<volatile unsigned long long *>(s_thrkey);
#pragma unroll 1
  for (int i = 0; i < Vec<BF16>::N; ++i) {
    const float xi = x[i];
    const unsigned long long key = make_key(xi, tok0 + i);
    bool inserted = false;
    if (xi == xi && key > tk) {
      unsigned long long carry = key;
      for (int s = 0; s < K; ++s) {
        unsigned long long old = atomicMax(&s_list[s], carry);
        if (old < carry) {
          carry = old;
          if (carry == 0ull) break;
        }
      }
      if (carry != key) {
        inserted = true;
        if (carry != 0ull) {
          acc_scalar(acc, key_value(carry));
          atomicMax(s_thrkey, carry);
        }
      }
      tk = *reinterpret_cast<volatile unsigned long long *>(s_thrkey);
    }
    if (!inserted) acc_scalar(acc, xi);
  }
  thr = key_value(tk);
}

template <bool BF16>
__device__ __forceinline__ void process_vector(uint4 q, int v, int K, Acc &acc, float &thr,
                                               unsigned long long *s_list,
                                               unsigned long long *s_thrkey) {
  Vec<BF16>::clamp(q);
  const float vm = Vec<BF16>::vmax(q);
  if (vm >= thr) slow_vector<BF16>(q, (uint32_t)v * Vec<BF16>::N, K, acc, thr, s_list, s_thrkey);
  else acc_vector<BF16>(acc, q);
}

template <bool BF16>
__global__ void __launch_bounds__(kPassThreads, kPassCtasPerSm) expand_pass_kernel(PassParams p) {
  using VT = Vec<BF16>;
  __shared__ int s_off[C2T_MAX_BATCH + 1];
  __shared__ unsigned long long s_list[C2T_MAX_TOPK];
  __shared__ unsigned long long s_thrkey;
  __shared__ uint32_t s_warm[kWarps * C2T_MAX_TOPK];
  __shared__ float s_mref0;
  __shared__ float s_red[kWarps][3];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int K = p.K;
  const int n_rows = build_row_offsets(p.counts, p.B, p.rows_per_seq_max, s_off);
  const Partition pt = make_partition<VT::N>(p, n_rows);
  if (pt.start >= pt.end) return;

  const size_t esz = BF16 ? 2 : 4;
  long long pos = pt.start;
  int a = (int)(pt.start / pt.vec_per_row);
  int v0 = (int)(pt.start - (long long)a * pt.vec_per_row);

  while (pos < pt.end) {
    const long long left = pt.end - pos;
    const int seg = left < (long long)(pt.vec_per_row - v0) ? (int)left : pt.vec_per_row - v0;
    const int v1 = v0 + seg;
    const int b = find_sequence(s_off, p.B, a);
    const int j = a - s_off[b];
    const char *row = reinterpret_cast<const char *>(p.logits) +
                      ((size_t)b * p.seq_stride + (size_t)j * p.row_stride) * esz;
    const int split = blockIdx.x - (int)(((long long)a * pt.vec_per_row) / pt.span);
    const size_t slot = (size_t)a * p.max_splits + split;

    // ---- warm-up: first vector of every thread seeds the filter and the reference
    int v = v0 + tid;
    uint4 q = make_uint4(0, 0, 0, 0);
    uint32_t u = f32_orderable(0xFF800000u);   // -inf
    const bool have_first = v < v1;
    if (have_first) {
      q = VT::load(row, v, pt.v_full, p.V);
      uint4 c = q;
      VT::clamp(c);
      float vm = VT::vmax(c);
      if (vm == vm) u = f32_orderable(__float_as_uint(vm));
    }
    {
      uint32_t live = u, mine = 0;
      for (int r = 0; r < K; ++r) {
        uint32_t mx = __reduce_max_sync(kFull, live);
        unsigned bal = __ballot_sync(kFull, live == mx);
        if (lane == __ffs(bal) - 1) live = 0;
        if (lane == r) mine = mx;
      }
      if (lane < K) s_warm[warp * K + lane] = mine;
    }
    __syncthreads();
    if (warp == 0) {
      constexpr int PER = (kWarps * C2T_MAX_TOPK) / 32;
      uint32_t vals[PER];
      const int n = kWarps * K;
#pragma unroll
      for (int i = 0; i < PER; ++i) {
        int idx = lane + 32 * i;
        vals[i] = idx < n ? s_warm[idx] : 0u;
      }
      uint32_t mx = 0, first = 0;
      for (int r = 0; r < K; ++r) {
        uint32_t lm = 0;
#pragma unroll
        for (int i = 0; i < PER; ++i) lm = vals[i] > lm ? vals[i] : lm;
        mx = __reduce_max_sync(kFull, lm);
        if (r == 0) first = mx;
        unsigned bal = __ballot_sync(kFull, lm == mx);
        if (lane == __ffs(bal) - 1) {
          bool done = false;
#pragma unroll
          for (int i = 0; i < PER; ++i)
            if (!done && vals[i] == mx) { vals[i] = 0; done = true; }
        }
      }
      if (lane < K) s_list[lane] = 0ull;
      if (lane == 0) {
        s_thrkey = (unsigned long long)mx << 32;
        s_mref0 = __uint_as_float(f32_from_orderable(first));
      }
    }
    __syncthreads();

    Acc acc;
    acc.m = s_mref0;
    acc.S0 = acc.S1 = acc.T0 = acc.T1 = 0.f;
    float thr = key_value(*reinterpret_cast<volatile unsigned long long *>(&s_thrkey));

    if (have_first) process_vector<BF16>(q, v, K, acc, thr, s_list, &s_thrkey);
    v += kPassThreads;
    for (; v + 3 * kPassThreads < v1; v += 4 * kPassThreads) {
      uint4 q0 = VT::load(row, v, pt.v_full, p.V);
      uint4 q1 = VT::load(row, v + kPassThreads, pt.v_full, p.V);
      uint4 q2 = VT::load(row, v + 2 * kPassThreads, pt.v_full, p.V);
      uint4 q3 = VT::load(row, v + 3 * kPassThreads, pt.v_full, p.V);
      thr = key_value(*reinterpret_cast<volatile unsigned long long *>(&s_thrkey));
      if (thr - acc.m > 60.f) acc_rescale(acc, thr);
      process_vector<BF16>(q0, v, K, acc, thr, s_list, &s_thrkey);
      process_vector<BF16>(q1, v + kPassThreads, K, acc, thr, s_list, &s_thrkey);
      process_vector<BF16>(q2, v + 2 * kPassThreads, K, acc, thr, s_list, &s_thrkey);
      process_vector<BF16>(q3, v + 3 * kPassThreads, K, acc, thr, s_list, &s_thrkey);
    }
    for (; v < v1; v += kPassThreads) {
      uint4 q0 = VT::load(row, v, pt.v_full, p.V);
      thr = key_value(*reinterpret_cast<volatile unsigned long long *>(&s_thrkey));
      if (thr - acc.m > 60.f) acc_rescale(acc, thr);
      process_vector<BF16>(q0, v, K, acc, thr, s_list, &s_thrkey);
    }

    // ---- segment end: merge the threads' sums, emit the partial record
    __syncthreads();
    float m = acc.m, S = acc.S0 + acc.S1, T = acc.T0 + acc.T1;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      float m2 = __shfl_down_sync(kFull, m, o);
      float S2 = __shfl_down_sync(kFull, S, o);
      float T2 = __shfl_down_sync(kFull, T, o);
      combine(m, S, T, m2, S2, T2);
    }
    if (lane == 0) { s_red[warp][0] = m; s_red[warp][1] = S; s_red[warp][2] = T; }
    __syncthreads();
    if (warp == 0) {
      if (lane < kWarps) { m = s_red[lane][0]; S = s_red[lane][1]; T = s_red[lane][2]; }
      else { m = s_red[0][0]; S = 0.f; T = 0.f; }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        float m2 = __shfl_down_sync(kFull, m, o);
        float S2 = __shfl_down_sync(kFull, S, o);
        float T2 = __shfl_down_sync(kFull, T, o);
        combine(m, S, T, m2, S2, T2);
      }
      // sort the list (descending, empty slots last) by counting
      unsigned long long mykey = lane < K ? s_list[lane] : 0ull;
      int rank = 0;
      for (int r = 0; r < K; ++r) {
        unsigned long long other = __shfl_sync(kFull, mykey, r);
        rank += (other > mykey) || (other == mykey && r < lane);
      }
      if (lane < K) p.part_keys[slot * K + rank] = mykey;
      unsigned nz = __ballot_sync(kFull, mykey != 0ull);
      if (lane == 0) p.part_stats[slot] = make_float4(m, S, T, __int_as_float(__popc(nz)));
    }
    pos += seg;
    ++a;
    v0 = 0;
  }
}

// ---------------------------------------------------------------- argmax ----

template <bool BF16>
__global__ void __launch_bounds__(kPassThreads, kPassCtasPerSm) argmax_pass_kernel(PassParams p) {
  using VT = Vec<BF16>;
  __shared__ int s_off[C2T_MAX_BATCH + 1];
  __shared__ unsigned long long s_best[kWarps];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n_rows = build_row_offsets(p.counts, p.B, p.rows_per_seq_max, s_off);
  const Partition pt = make_partition<VT::N>(p, n_rows);
  if (pt.start >= pt.end) return;

  const size_t esz = BF16 ? 2 : 4;
  long long pos = pt.start;
  int a = (int)(pt.start / pt.vec_per_row);
  int v0 = (int)(pt.start - (long long)a * pt.vec_per_row);

  while (pos < pt.end) {
    const long long left = pt.end - pos;
    const int seg = left < (long long)(pt.vec_per_row - v0) ? (int)left : pt.vec_per_row - v0;
    const int v1 = v0 + seg;
    const int b = find_sequence(s_off, p.B, a);
    const int j = a - s_off[b];
    const char *row = reinterpret_cast<const char *>(p.logits) +
                      ((size_t)b * p.seq_stride + (size_t)j * p.row_stride) * esz;
    const int split = blockIdx.x - (int)(((long long)a * pt.vec_per_row) / pt.span);
    const size_t slot = (size_t)a * p.max_splits + split;

    float m = -INFINITY;   // clamped values are finite, so any non-NaN vector beats this
    int mv = -1;
    int v = v0 + tid;
    for (; v + 3 * kPassThreads < v1; v += 4 * kPassThreads) {
      uint4 q[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) q[i] = VT::load(row, v + i * kPassThreads, pt.v_full, p.V);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        VT::clamp(q[i]);
        float vm = VT::vmax(q[i]);
        if (vm > m) { m = vm; mv = v + i * kPassThreads; }
      }
    }
    for (; v < v1; v += kPassThreads) {
      uint4 q = VT::load(row, v, pt.v_full, p.V);
      VT::clamp(q);
      float vm = VT::vmax(q);
      if (vm > m) { m = vm; mv = v; }
    }
    unsigned long long best = 0ull;
    if (mv >= 0) {
      uint4 q = VT::load(row, mv, pt.v_full, p.V);
      VT::clamp(q);
      float x[VT::N];
      VT::unpack(q, x);
#pragma unroll
      for (int i = VT::N - 1; i >= 0; --i)
        if (x[i] == m && mv * VT::N + i < p.V) best = make_key(m, (uint32_t)(mv * VT::N + i));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      unsigned long long other = __shfl_down_sync(kFull, best, o);
      best = other > best ? other : best;
    }
    if (lane == 0) s_best[warp] = best;
    __syncthreads();
    if (warp == 0) {
      best = lane < kWarps ? s_best[lane] : 0ull;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        unsigned long long other = __shfl_down_sync(kFull, best, o);
        best = other > best ? other : best;
      }
      if (lane == 0) p.part_best[slot] = best;
    }
    __syncthreads();
    pos += seg;
    ++a;
    v0 = 0;
  }
}

}  // namespace

int max_splits_for(int vocab, int elem_bytes, int grid) {
  const int vec = 16 / elem_bytes;
  const int vec_per_row = (vocab + vec - 1) / vec;
  int by_span = (vec_per_row + kMinSpanVectors - 1) / kMinSpanVectors;
  if (by_span > grid) by_span = grid;
  return by_span + 1;
}

cudaError_t launch_expand_pass(const PassParams &p, int dtype, int grid, cudaStream_t s) {
  if (dtype == C2T_BF16) expand_pass_kernel<true><<<grid, kPassThreads, 0, s>>>(p);
  else expand_pass_kernel<false><<<grid, kPassThreads, 0, s>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_argmax_pass(const PassParams &p, int dtype, int grid, cudaStream_t s) {
  if (dtype == C2T_BF16) argmax_pass_kernel<true><<<grid, kPassThreads, 0, s>>>(p);
  else argmax_pass_kernel<false><<<grid, kPassThreads, 0, s>>>(p);
  return cudaGetLastError();
}

}  // namespace c2t
