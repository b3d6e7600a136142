// Truncated entropy (Eq. 3): the sums over the M most probable tokens of every active draft row,
// for configurations with entropy_top_m = M > 0.  The probabilities are those of the full softmax
// (no renormalisation), so the expand pass still supplies the normaliser; this pass supplies
//     S_M = sum over the top M of e^(x - m),   T_M = sum over the top M of e^(x - m) (x - m)
// (m = the row maximum), from which  H_M = (ln Z * S_M - T_M) / Z.
//
// One CTA per active row.  The M-th largest value is found by a radix select on the order-
// preserving 32-bit image of the values, one byte per step from the top (two steps for bf16,
// whose images differ in the upper 16 bits only; four for fp32); then the terms above that
// value are added, and as many copies of the term AT that value as are still missing (equal
// values give equal terms, so which tokens are taken does not matter).
//   Fast path: the row maximum is known from the expand pass, which runs just before; one sweep
// copies the elements within two top key bytes of it to shared memory and everything else runs
// on those.  General path (the guess failed): up to five sweeps over the row, which stays in L2;
// the top byte is counted in registers from the maximum's bin downwards, the later bytes with a
// 256-bin histogram in shared memory over the elements that still match.
// An optional mode, not tuned further: about 2.4 times the expand pass on a 640-row level.
#include "vocab_common.cuh"

namespace c2t {
namespace {

#ifndef C2T_TOPM_THREADS
#define C2T_TOPM_THREADS 1024
#define C2T_TOPM_CAND 32768
#endif
constexpr int kTopmThreads = C2T_TOPM_THREADS;
constexpr int kTopmBatch = 8;          // independent 16-byte loads a thread keeps in flight
constexpr int kTopmCand = C2T_TOPM_CAND;   // candidate keys the fast path can hold in shared memory

// Where the expand pass, which runs just before, left what this pass can reuse: the row's maximum
// is the largest of the keys held out of its partial sums.
struct TopmAux {
  const unsigned long long *part_held;
  const PassInfo *info;
  const int32_t *row_off;
  int max_splits;
};

// The bin, from 255 downwards, in which the need-th largest counted element lies, and how many
// elements the bins above it hold.  Called by warp 0; lane l owns bins 8l .. 8l+7.
__device__ __forceinline__ void select_bin(const unsigned *hist, unsigned need, int &bin, unsigned &above) {
  const int lane = threadIdx.x & 31;
  unsigned h[8], mine = 0u;
#pragma unroll
  for (int i = 0; i < 8; ++i) { h[i] = hist[lane * 8 + i]; mine += h[i]; }
  unsigned suf = mine;                                 // inclusive suffix sum over the lanes: bins 8*lane and up
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned v = __shfl_down_sync(kFull, suf, o);
    if (lane + o < 32) suf += v;
  }
  const unsigned higher = suf - mine;                  // elements in the bins of higher lanes
  const bool here = higher < need && suf >= need;      // exactly one lane, unless fewer than need were counted
  const unsigned owner = __ballot_sync(kFull, here);
  int b_sel = 0;
  unsigned a_sel = 0u;
  if (here) {
    unsigned acc = higher;
    b_sel = lane * 8;
    a_sel = acc;
#pragma unroll
    for (int i = 7; i >= 0; --i) {
      if (acc + h[i] >= need) { b_sel = lane * 8 + i; a_sel = acc; break; }
      acc += h[i];
    }
  }
  const int src = owner ? __ffs(owner) - 1 : 0;        // no owner: everything counted is wanted, bin 0
  bin = __shfl_sync(kFull, b_sel, src);
  above = __shfl_sync(kFull, a_sel, src);
  if (!owner) { bin = 0; above = __shfl_sync(kFull, suf, 0) - hist[0]; }
}

template <bool BF16>
__global__ void __launch_bounds__(kTopmThreads) topm_entropy_kernel(const void *logits, long long seq_stride,
                                                                    long long row_stride, int V, int M, int F,
                                                                    const int32_t *counts, TopmAux aux, double2 *out) {
  extern __shared__ uint32_t s_cand[];             // kTopmCand keys of the fast path
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

  using VT = Vec<BF16>;
  const int vpr = (V + VT::N - 1) / VT::N, v_full = V / VT::N;
  const int sweeps = (vpr + kTopmThreads - 1) / kTopmThreads;     // the same trip count for every thread
  const uint32_t lo = BF16 ? kLowestBf16x2 : __float_as_uint(kLowestF32);

  // ---- fast path: ONE sweep.  The maximum is known from the expand pass; the M-th largest value
  // almost always lies within two top key bytes below the maximum's (a factor 64 to 256 in value), so
  // the elements from there upwards are copied to shared memory and the selection runs on them alone;
  // rows where that guess fails (fewer than M such elements, or more than fit) take the general path.
  if (M < V) {
    const PassInfo info = *aux.info;
    const int a = aux.row_off[b] + j;
    const long long first_vec = (long long)a * (info.vec_per_row + info.pad) + info.pad;
    const int c_first = (int)(first_vec / info.span);
    int n_splits = (int)((first_vec + info.vec_per_row - 1) / info.span) - c_first + 1;
    if (n_splits > aux.max_splits) n_splits = aux.max_splits;
    unsigned long long top = 0ull;
    for (int sp = 0; sp < n_splits; ++sp) {
      const unsigned long long k = aux.part_held[(size_t)a * aux.max_splits + sp];
      top = k > top ? k : top;
    }
    const uint32_t top_key = (uint32_t)(top >> 32);
    const int d0 = (int)(top_key >> 24);
    const float mf = key_value(top);
    if (tid == 0) { s_win[0] = 0u; s_win[1] = 0u; s_found = 0; }
    __syncthreads();
    const float floor1 = __uint_as_float(f32_from_orderable((uint32_t)(d0 >= 2 ? d0 - 2 : 0) << 24));   // smallest value of byte d0-2
    // (uniform; the floor must stay above -2^127, the value that pads a ragged vector)
    if (top != 0ull && d0 >= 2 && mf < INFINITY && floor1 > kLowestF32) {
      for (int it0 = 0; it0 < sweeps; it0 += kTopmBatch) {
        uint4 qb[kTopmBatch];
#pragma unroll
        for (int k = 0; k < kTopmBatch; ++k) {
          const int vec = (it0 + k) * kTopmThreads + tid;
          qb[k] = vec < vpr ? VT::load(row, vec, v_full, V) : make_uint4(lo, lo, lo, lo);
        }
#pragma unroll
        for (int k = 0; k < kTopmBatch; ++k) {
          VT::clamp(qb[k]);
          if (!__any_sync(kFull, VT::vmax(qb[k]) >= floor1)) continue;
          float x[VT::N];
          VT::unpack(qb[k], x);
          // one reservation per warp and vector: lane counts, warp prefix sum, one atomic
          unsigned cnt = 0u;
#pragma unroll
          for (int i = 0; i < VT::N; ++i) cnt += x[i] >= floor1;     // false for NaN and for a ragged vector's padding
          unsigned inc = cnt;
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const unsigned v = __shfl_up_sync(kFull, inc, o);
            if (lane >= o) inc += v;
          }
          unsigned base = 0u;
          if (lane == 31) base = atomicAdd(&s_win[1], inc);
          unsigned pos = __shfl_sync(kFull, base, 31) + inc - cnt;
#pragma unroll
          for (int i = 0; i < VT::N; ++i)
            if (x[i] >= floor1) {
              if (pos < (unsigned)kTopmCand) s_cand[pos] = f32_orderable(__float_as_uint(x[i]));
              ++pos;
            }
        }
      }
      __syncthreads();
      const unsigned n_c = s_win[1];
      if (n_c >= (unsigned)M && n_c <= (unsigned)kTopmCand) {                     // (uniform)
        // radix select of the M-th largest among the candidates
        if (tid == 0) { s_prefix = 0u; s_need = (unsigned)M; }
        const int steps_f = BF16 ? 2 : 4;
        for (int st = 0; st < steps_f; ++st) {
          const int shift = 24 - 8 * st;
          for (int i = tid; i < 256; i += kTopmThreads) s_hist[i] = 0u;
          __syncthreads();
          const unsigned prefix = s_prefix;
          for (unsigned i = tid; i < n_c; i += kTopmThreads) {
            const uint32_t key = s_cand[i];
            if (st == 0 || (key >> (shift + 8)) == (prefix >> (shift + 8))) atomicAdd(&s_hist[(key >> shift) & 255u], 1u);
          }
          __syncthreads();
          if (warp == 0) {
            int d;
            unsigned above;
            const unsigned need = s_need;
            select_bin(s_hist, need, d, above);
            __syncwarp();
            if (lane == 0) { s_need = need - above; s_prefix = prefix | ((unsigned)d << shift); }
          }
          __syncthreads();
        }
        const uint32_t tmask = BF16 ? 0xFFFF0000u : 0xFFFFFFFFu;
        const uint32_t tau_f = s_prefix & tmask;
        double Sd = 0.0, Td = 0.0;
        for (unsigned i = tid; i < n_c; i += kTopmThreads) {
          const uint32_t key = s_cand[i];
          if ((key & tmask) > tau_f) {
            const float d = __uint_as_float(f32_from_orderable(key)) - mf;
            const float e = expf(d);
            Sd += (double)e;
            Td += (double)(e * d);
          }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          Sd += __shfl_xor_sync(kFull, Sd, o);
          Td += __shfl_xor_sync(kFull, Td, o);
        }
        if (lane == 0) { s_sum[0][warp] = Sd; s_sum[1][warp] = Td; }
        __syncthreads();
        if (tid == 0) {
          double St = 0.0, Tt = 0.0;
          for (int w = 0; w < kTopmThreads / 32; ++w) { St += s_sum[0][w]; Tt += s_sum[1][w]; }
          const unsigned need = s_need;
          const uint32_t tk = BF16 ? tau_f | ((tau_f >> 31) ? 0u : 0xFFFFu) : tau_f;
          const double d = (double)__uint_as_float(f32_from_orderable(tk)) - (double)mf;
          const double e = exp(d);
          St += (double)need * e;
          Tt += (double)need * e * d;
          out[(size_t)b * F + j] = make_double2(St, Tt);
        }
        return;
      }
    }
    __syncthreads();
  }

  // ---- general path: the row maximum (NaN elements ignored; a row with NaN is reported by the expand pass)
  float m = -INFINITY;
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
    // The M-th largest can lie far below the maximum's bin (a positive maximum and a negative M-th largest are half
    // the key space apart): one sweep over the top four key bits first, so that the fine count starts at most
    // sixteen bins above its goal.
    if (tid < 16) s_hist[tid] = 0u;
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
          unsigned bin = 0xFFFFFFFFu;
          if (vec < vpr && vec * VT::N + i < V && x[i] == x[i]) bin = f32_orderable(__float_as_uint(x[i])) >> 28;
          const unsigned peers = __match_any_sync(kFull, bin);
          if (bin != 0xFFFFFFFFu && lane == __ffs(peers) - 1) atomicAdd(&s_hist[bin], (unsigned)__popc(peers));
        }
      }
    }
    __syncthreads();
    if (tid == 0) {
      unsigned need = s_need;
      int cb = 15;
      for (; cb > 0 && s_hist[cb] < need; --cb) need -= s_hist[cb];
      s_need = need;                               // still wanted from coarse bin cb downwards
      s_found = cb;
    }
    __syncthreads();
    {
      const int top_of_coarse = s_found * 16 + 15;
      d0 = d0 < top_of_coarse ? d0 : top_of_coarse;
    }
    __syncthreads();
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
    if (warp == 0) {                           // the bin that holds the need-th largest of the matching elements
      int d;
      unsigned above;
      const unsigned need = s_need;
      select_bin(s_hist, need, d, above);
      __syncwarp();
      if (lane == 0) { s_need = need - above; s_prefix = prefix | ((unsigned)d << shift); }   // still wanted from bin d
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

static size_t topm_dynamic_smem() { return (size_t)kTopmCand * sizeof(uint32_t); }

cudaError_t prepare_topm_pass() {
  const int bytes = (int)topm_dynamic_smem();
  cudaError_t e = cudaFuncSetAttribute(topm_entropy_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(topm_entropy_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
}

cudaError_t launch_topm_entropy(const void *logits, int64_t seq_stride, int64_t row_stride, int V, int M, int F,
                                int B, const int32_t *counts, const TreeState &t, double2 *out, int dtype,
                                cudaStream_t s) {
  const dim3 grid(F, B);
  TopmAux aux;
  aux.part_held = t.part_held; aux.info = t.info_draft; aux.row_off = t.row_off_draft; aux.max_splits = t.max_splits;
  const size_t smem = topm_dynamic_smem();
  if (dtype == C2T_BF16)
    topm_entropy_kernel<true><<<grid, kTopmThreads, smem, s>>>(logits, seq_stride, row_stride, V, M, F, counts, aux, out);
  else
    topm_entropy_kernel<false><<<grid, kTopmThreads, smem, s>>>(logits, seq_stride, row_stride, V, M, F, counts, aux, out);
  return cudaGetLastError();
}

}  // namespace c2t
