// Truncated entropy (Eq. 3): the sums over the M most probable tokens of every active draft row,
// for configurations with entropy_top_m = M > 0.  The probabilities are those of the full softmax
// (no renormalisation), so the expand pass still supplies the normaliser; this pass supplies
//     S_M = sum over the top M of e^(x - m),   T_M = sum over the top M of e^(x - m) (x - m)
// (m = the row maximum), from which  H_M = (ln Z * S_M - T_M) / Z.
//
// One CTA per active row.  The M-th largest value is found by a radix select on the order-
// preserving 32-bit image of the values, one byte per step from the top (two steps for bf16,
// whose images differ in the upper 16 bits only; four for fp32): the top byte by counting the
// few bins below the maximum's in registers, the later bytes with a 256-bin histogram in shared
// memory over the elements that match so far; then one more sweep adds the terms above that value and as many copies of the
// term AT that value as are still missing (equal values give equal terms, so which tokens are
// taken does not matter).  The row (at most 1 MB) is re-read from L2 by the later sweeps.  This is an
// optional mode and is not tuned: it costs about one more pass over the logits.
#include "vocab_common.cuh"

namespace c2t {
namespace {

constexpr int kTopmThreads = 1024;
constexpr int kTopmBatch = 4;          // independent 16-byte loads a thread keeps in flight

template <bool BF16>
__global__ void __launch_bounds__(kTopmThreads) topm_entropy_kernel(const void *logits, long long seq_stride,
                                                                    long long row_stride, int V, int M, int F,
                                                                    const int32_t *counts, double2 *out) {
  __shared__ unsigned s_hist[256];
  __shared__ float s_red[kTopmThreads / 32];
  __shared__ double s_sum[2][kTopmThreads / 32];
  __shared__ unsigned s_prefix, s_need, s_win[4];
  __shared__ int s_found;
  const int b = blockIdx.y, j = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  int n = counts[b];
  n = n < 0 ? 0 : (n > F ? F : n);
  if (j >= n) return;
  const size_t esz = BF16 ? 2 : 4;
  const char *row = reinterpret_cast<const char *>(logits) + ((size_t)b * seq_stride + (size_t)j * row_stride) * esz;

  // the row maximum (NaN elements ignored; a row with NaN is reported by the expand pass)
  using VT = Vec<BF16>;
  const int vpr = (V + VT::N - 1) / VT::N, v_full = V / VT::N;
  const int sweeps = (vpr + kTopmThreads - 1) / kTopmThreads;     // the same trip count for every thread
  float m = -INFINITY;
  const uint32_t lo = BF16 ? kLowestBf16x2 : __float_as_uint(kLowestF32);
  for (int it = 0; it < sweeps; it += kTopmBatch) {
    uint4 q[kTopmBatch];
#pragma unroll
    for (int k = 0; k < kTopmBatch; ++k) {        // 16 bytes each; a ragged last vector is padded with the lowest value
      const int vec = (it + k) * kTopmThreads + tid;
      q[k] = vec < vpr ? VT::load(row, vec, v_full, V) : make_uint4(lo, lo, lo, lo);
    }
#pragma unroll
    for (int k = 0; k < kTopmBatch; ++k) {
      VT::clamp(q[k]);
      const float vm = VT::vmax(q[k]);
      if (vm == vm) m = fmaxf(m, vm);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(kFull, m, o));
  if (lane == 0) s_red[warp] = m;
  if (tid == 0) { s_prefix = 0u; s_need = (unsigned)M; }
  __syncthreads();
  m = s_red[0];
  // (clamped values are finite, so m is finite unless the row holds only NaN)
  for (int w = 1; w < kTopmThreads / 32; ++w) m = fmaxf(m, s_red[w]);

  // radix select of the M-th largest key among the V elements (every element if M >= V)
  const bool all = M >= V;
  const int steps = BF16 ? 2 : 4;
  // Step 0 (top byte) counts in registers: the M-th largest sits a few bins below the maximum's, so the
  // bins are visited four at a time from there downwards and the bulk of the row is never counted.
  if (!all) {
    int d0 = (int)(f32_orderable(__float_as_uint(m)) >> 24);
    for (;;) {
      unsigned c[4] = {0u, 0u, 0u, 0u};
      if (tid < 4) s_win[tid] = 0u;
      __syncthreads();
      for (int it0 = 0; it0 < sweeps; it0 += kTopmBatch) {
        uint4 qb[kTopmBatch];
#pragma unroll
        for (int k = 0; k < kTopmBatch; ++k) {
          const int vec = (it0 + k) * kTopmThreads + tid;
          qb[k] = vec < vpr ? VT::load(row, vec, v_full, V) : make_uint4(lo, lo, lo, lo);
        }
#pragma unroll
        for (int k = 0; k < kTopmBatch; ++k) {
          const int vec = (it0 + k) * kTopmThreads + tid;
          float x[VT::N];
          VT::clamp(qb[k]);
          VT::unpack(qb[k], x);
#pragma unroll
          for (int i = 0; i < VT::N; ++i) {
            if (vec >= vpr || vec * VT::N + i >= V || x[i] != x[i]) continue;
            const int tb = (int)(f32_orderable(__float_as_uint(x[i])) >> 24);
#pragma unroll
            for (int w = 0; w < 4; ++w) c[w] += tb == d0 - w;
          }
        }
      }
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        unsigned v = c[w];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
        if (lane == 0 && v) atomicAdd(&s_win[w], v);
      }
      __syncthreads();
      if (tid == 0) {
        unsigned need = s_need;
        int found = -1;
        for (int w = 0; w < 4 && found < 0; ++w) {
          if (s_win[w] >= need || d0 - w <= 0) found = d0 - w < 0 ? 0 : d0 - w;
          else need -= s_win[w];
        }
        s_need = need;
        s_found = found;
        if (found >= 0) s_prefix = (unsigned)found << 24;
      }
      __syncthreads();
      if (s_found >= 0) break;
      d0 -= 4;
    }
  }
  for (int s = 1; s < steps && !all; ++s) {
    const int shift = 24 - 8 * s;
    for (int i = tid; i < 256; i += kTopmThreads) s_hist[i] = 0u;
    __syncthreads();
    const unsigned prefix = s_prefix;
    const float prefix_floor = __uint_as_float(f32_from_orderable(prefix));
    for (int it0 = 0; it0 < sweeps; it0 += kTopmBatch) {
      uint4 qb[kTopmBatch];
#pragma unroll
      for (int k = 0; k < kTopmBatch; ++k) {
        const int vec = (it0 + k) * kTopmThreads + tid;
        qb[k] = vec < vpr ? VT::load(row, vec, v_full, V) : make_uint4(lo, lo, lo, lo);
      }
#pragma unroll
      for (int k = 0; k < kTopmBatch; ++k) {
      const int vec = (it0 + k) * kTopmThreads + tid;
      float x[VT::N];
      VT::clamp(qb[k]);
      // nothing in most vectors reaches the smallest value with this prefix (warp-uniform skip)
      if (!__any_sync(kFull, VT::vmax(qb[k]) >= prefix_floor)) continue;
      VT::unpack(qb[k], x);
#pragma unroll
      for (int i = 0; i < VT::N; ++i) {
        // most elements share a few bins: the lanes of a warp that hit the same bin add once
        unsigned bin = 0xFFFFFFFFu;
        if (vec < vpr && vec * VT::N + i < V && x[i] == x[i]) {
          const uint32_t key = f32_orderable(__float_as_uint(x[i]));
          if ((key >> (shift + 8)) == (prefix >> (shift + 8))) bin = (key >> shift) & 255u;
        }
        const unsigned peers = __match_any_sync(kFull, bin);
        if (bin != 0xFFFFFFFFu && lane == __ffs(peers) - 1) atomicAdd(&s_hist[bin], (unsigned)__popc(peers));
      }
      }
    }
    __syncthreads();
    if (tid == 0) {
      unsigned need = s_need, above = 0u;
      int d = 255;
      for (; d > 0; --d) {                     // the bin that holds the need-th largest of the matching elements
        if (above + s_hist[d] >= need) break;
        above += s_hist[d];
      }
      s_need = need - above;                   // how many are still wanted from bin d
      s_prefix = prefix | ((unsigned)d << shift);
    }
    __syncthreads();
  }
  // keys above tau are all taken; of the keys equal to tau, `need` are
  const uint32_t tau = all ? 0u : s_prefix;
  const uint32_t tau_mask = BF16 ? 0xFFFF0000u : 0xFFFFFFFFu;   // bf16 images are told apart by the upper half
  const unsigned need = all ? 0u : s_need;
  const float tau_floor = __uint_as_float(f32_from_orderable(tau & tau_mask));   // at or below the M-th largest value

  double S = 0.0, T = 0.0;
  float S32 = 0.f, T32 = 0.f;
  int since = 0;
  for (int it0 = 0; it0 < sweeps; it0 += kTopmBatch) {
    uint4 qb[kTopmBatch];
#pragma unroll
    for (int k = 0; k < kTopmBatch; ++k) {
      const int vec = (it0 + k) * kTopmThreads + tid;
      qb[k] = vec < vpr ? VT::load(row, vec, v_full, V) : make_uint4(lo, lo, lo, lo);
    }
#pragma unroll
    for (int k = 0; k < kTopmBatch; ++k) {
    const int vec = (it0 + k) * kTopmThreads + tid;
    if (vec >= vpr) continue;
    VT::clamp(qb[k]);
    if (!all && !(VT::vmax(qb[k]) >= tau_floor)) continue;     // no element of this vector is among the top M
    float x[VT::N];
    VT::unpack(qb[k], x);
#pragma unroll
    for (int i = 0; i < VT::N; ++i) {
      if (vec * VT::N + i >= V || x[i] != x[i]) continue;
      const uint32_t key = f32_orderable(__float_as_uint(x[i])) & tau_mask;
      if (all || key > (tau & tau_mask)) {
        const float d = x[i] - m;
        const float e = expf(d);
        S32 += e;
        T32 = fmaf(e, d, T32);
        if (++since == 64) { S += (double)S32; T += (double)T32; S32 = T32 = 0.f; since = 0; }   // short fp32 runs
      }
    }
    }
  }
  S += (double)S32; T += (double)T32;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    S += __shfl_xor_sync(kFull, S, o);
    T += __shfl_xor_sync(kFull, T, o);
  }
  if (lane == 0) { s_sum[0][warp] = S; s_sum[1][warp] = T; }
  __syncthreads();
  if (tid == 0) {
    double St = 0.0, Tt = 0.0;
    for (int w = 0; w < kTopmThreads / 32; ++w) { St += s_sum[0][w]; Tt += s_sum[1][w]; }
    if (!all && need > 0u) {
      const float xt = __uint_as_float(f32_from_orderable(BF16 ? (tau & tau_mask) | ((tau >> 31) ? 0u : 0xFFFFu) : tau));
      const double d = (double)xt - (double)m;
      const double e = exp(d);
      St += (double)need * e;
      Tt += (double)need * e * d;
    }
    out[(size_t)b * F + j] = make_double2(St, Tt);
  }
}

}  // namespace

cudaError_t launch_topm_entropy(const void *logits, int64_t seq_stride, int64_t row_stride, int V, int M, int F,
                                int B, const int32_t *counts, double2 *out, int dtype, cudaStream_t s) {
  const dim3 grid(F, B);
  if (dtype == C2T_BF16)
    topm_entropy_kernel<true><<<grid, kTopmThreads, 0, s>>>(logits, seq_stride, row_stride, V, M, F, counts, out);
  else
    topm_entropy_kernel<false><<<grid, kTopmThreads, 0, s>>>(logits, seq_stride, row_stride, V, M, F, counts, out);
  return cudaGetLastError();
}

}  // namespace c2t
