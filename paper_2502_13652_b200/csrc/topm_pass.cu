// Truncated entropy (Eq. 3): the sums over the M most probable tokens of every active draft row,
// for configurations with entropy_top_m = M > 0.  The probabilities are those of the full softmax
// (no renormalisation), so the expand pass still supplies the normaliser; the kernels here supply
//     S_M = sum over the top M of e^(x - m),   T_M = sum over the top M of e^(x - m) (x - m)
// (m = the row maximum), from which  H_M = (ln Z * S_M - T_M) / Z.
//
// In both kernels the M-th largest value of a row is found on the order-preserving 32-bit image of
// the values; then the terms above that value are added, and as many copies of the term AT that
// value as are still missing (equal values give equal terms, so which tokens are taken does not
// matter).
//   topm_finish_kernel, one CTA per active row, works on the vectors that the expand pass set aside
// (every vector with an element at or above a per-segment floor): if at least M elements reach the
// highest floor among the row's segments, the M largest are among them.  The rows are not read again.
//   topm_entropy_kernel, a persistent grid, takes the rows that kernel could not serve and reads them
// once more.  Fast path: the row maximum is known from the expand pass; one sweep copies the elements
// within two top key bytes of it to shared memory and the selection runs on those.  General path (that
// guess failed too): a radix select over the row in up to five sweeps (the row stays in L2); the top
// byte is counted in registers from the maximum's bin downwards, the later bytes with a 256-bin
// histogram in shared memory over the elements that still match.
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

// The elements of a vector at or above a floor, as keys, appended to a candidate set in shared memory (called by whole
// warps: one reservation per warp and vector).  The count keeps rising when the set is full.
template <bool BF16>
__device__ __forceinline__ void push_candidates(const uint4 &q, float floor, uint32_t *s_cand, unsigned cap, unsigned *s_count) {
  using VT = Vec<BF16>;
  const int lane = threadIdx.x & 31;
  float x[VT::N];
  VT::unpack(q, x);
  unsigned cnt = 0u;
#pragma unroll
  for (int i = 0; i < VT::N; ++i) cnt += x[i] >= floor;        // false for NaN and for a ragged vector's padding
  unsigned inc = cnt;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned v = __shfl_up_sync(kFull, inc, o);
    if (lane >= o) inc += v;
  }
  unsigned base = 0u;
  if (lane == 31) base = atomicAdd(s_count, inc);
  unsigned pos = __shfl_sync(kFull, base, 31) + inc - cnt;
#pragma unroll
  for (int i = 0; i < VT::N; ++i)
    if (x[i] >= floor) {
      if (pos < cap) s_cand[pos] = f32_orderable(__float_as_uint(x[i]));
      ++pos;
    }
}

// Eq. 3's sums from a candidate set in shared memory that is known to hold the M largest elements of the row
// (n_c >= M keys, the order-preserving images of the values): the M-th largest key, then the terms above it and as
// many copies of the term at it as are still missing.  Called by all NT threads of the CTA; thread 0 writes the
// result.
//   The candidates lie close together (between a floor and the row maximum), so a histogram over fixed key bytes
// would put nearly all of them in one bin, one shared-memory atomic after the other.  The bins follow the data
// instead: kSelBins equal steps between the smallest and the largest key still in play, refined until a step is
// one key wide (one round for bf16 rows as a rule, two or three for fp32).
constexpr int kSelBins = 2048;

// key_lo, key_hi: keys that bound the set from below and from above (the floor it was collected with, the row maximum).
template <bool BF16, int NT>
__device__ __forceinline__ void select_and_sum(const uint32_t *s_cand, unsigned n_c, int M, float mf, uint32_t key_lo,
                                               uint32_t key_hi, double *s_sum, unsigned *s_need, double2 *out) {
  __shared__ unsigned s_bins[kSelBins];
  __shared__ unsigned s_wsum[NT / 32], s_lo, s_hi;
  __shared__ double s_tail[2];
  constexpr int BPT = kSelBins / NT;               // bins a thread owns when the bin with the M-th largest is looked for
  static_assert(kSelBins % NT == 0, "whole bins per thread");
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int KS = BF16 ? 16 : 0;                // bf16 images are told apart by their upper halves
  if (key_lo == 0x80000000u) key_lo = 0x7FFFFFFFu; // a floor of +0 also admits -0, whose key is one lower
  if (tid == 0) { s_lo = key_lo >> KS; s_hi = key_hi >> KS; *s_need = (unsigned)M; }
  __syncthreads();
  // ---- refine [lo, hi] around the M-th largest key
  for (int round = 0; round < 4; ++round) {          // (32 key bits, 11 per round: three at most)
    const uint32_t lo = s_lo, hi = s_hi;
    const unsigned need = *s_need;
    if (lo == hi) break;                             // (uniform) one key left: `need` copies of it are still missing
    const uint32_t range = hi - lo;
    const int shift = range < (uint32_t)kSelBins ? 0 : 32 - __clz(range) - 11;     // range >> shift < kSelBins
    for (int i = tid; i < kSelBins; i += NT) s_bins[i] = 0u;
    __syncthreads();
    for (unsigned i = tid; i < n_c; i += NT) {
      const uint32_t k = s_cand[i] >> KS;
      if (k >= lo && k <= hi) atomicAdd(&s_bins[(k - lo) >> shift], 1u);
    }
    __syncthreads();
    // the bin, from the top, that holds the need-th largest: thread t owns bins [t BPT, (t + 1) BPT)
    unsigned h[BPT], mine = 0u;
#pragma unroll
    for (int i = 0; i < BPT; ++i) { h[i] = s_bins[tid * BPT + i]; mine += h[i]; }
    unsigned suf = mine;                             // inclusive suffix sum over the lanes of the warp
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned v = __shfl_down_sync(kFull, suf, o);
      if (lane + o < 32) suf += v;
    }
    if (lane == 0) s_wsum[warp] = suf;
    __syncthreads();
    unsigned higher = suf - mine;                    // keys in the bins of higher threads
    for (int w = warp + 1; w < NT / 32; ++w) higher += s_wsum[w];
    if (higher < need && higher + mine >= need) {    // exactly one thread (at least `need` keys are in play)
      unsigned acc = higher;
      int d = tid * BPT;
#pragma unroll
      for (int i = BPT - 1; i >= 0; --i) {
        if (acc + h[i] >= need) { d = tid * BPT + i; break; }
        acc += h[i];
      }
      const uint32_t new_lo = lo + ((uint32_t)d << shift);
      const uint32_t step_top = new_lo + ((1u << shift) - 1u);
      s_lo = new_lo;
      s_hi = step_top < hi ? step_top : hi;
      *s_need = need - acc;
    }
    __syncthreads();
    if (shift == 0) break;                           // (uniform) the bin was one key
  }
  // keys above tau are all taken; of the keys equal to tau, *s_need are
  const uint32_t tau = s_lo;
  double Sd = 0.0, Td = 0.0;
  for (unsigned i = tid; i < n_c; i += NT) {
    const uint32_t key = s_cand[i];
    if ((key >> KS) > tau) {
      const float d = __uint_as_float(f32_from_orderable(key)) - mf;
      const float e = ex2f(d * kLog2e);            // (the expand pass takes its exponentials the same way)
      Sd += (double)e;
      Td += (double)(e * d);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    Sd += __shfl_xor_sync(kFull, Sd, o);
    Td += __shfl_xor_sync(kFull, Td, o);
  }
  if (lane == 0) { s_sum[warp] = Sd; s_sum[NT / 32 + warp] = Td; }
  if (tid == NT - 1) {                               // meanwhile: the term at tau (its double-precision exp is long)
    // the key's value (a bf16 image's lower half is all ones for a negative value)
    const uint32_t tk = BF16 ? (tau << 16) | ((tau >> 15) ? 0u : 0xFFFFu) : tau;
    const double d = (double)__uint_as_float(f32_from_orderable(tk)) - (double)mf;
    const double e = exp(d);
    s_tail[0] = e;
    s_tail[1] = e * d;
  }
  __syncthreads();
  if (tid == 0) {
    double St = 0.0, Tt = 0.0;
    for (int w = 0; w < NT / 32; ++w) { St += s_sum[w]; Tt += s_sum[NT / 32 + w]; }
    const unsigned need = *s_need;
    St += (double)need * s_tail[0];
    Tt += (double)need * s_tail[1];
    *out = make_double2(St, Tt);
  }
}

// One row, by all threads of a CTA (s_cand: kTopmCand keys of the fast path).
template <bool BF16>
__device__ __forceinline__ void topm_entropy_row(const void *logits, long long seq_stride, long long row_stride, int V,
                                                 int M, int F, const TopmAux &aux, double2 *out, int b, int j,
                                                 uint32_t *s_cand) {
  __shared__ unsigned s_hist[256];
  __shared__ float s_red[kTopmThreads / 32];
  __shared__ double s_sum[2 * (kTopmThreads / 32)];
  __shared__ unsigned s_prefix, s_need, s_win[4];
  __shared__ int s_found;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
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
          push_candidates<BF16>(qb[k], floor1, s_cand, (unsigned)kTopmCand, &s_win[1]);
        }
      }
      __syncthreads();
      const unsigned n_c = s_win[1];
      if (n_c >= (unsigned)M && n_c <= (unsigned)kTopmCand) {                     // (uniform)
        select_and_sum<BF16, kTopmThreads>(s_cand, n_c, M, mf, f32_orderable(__float_as_uint(floor1)), top_key, s_sum, &s_need,
                                           &out[(size_t)b * F + j]);
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
  if (lane == 0) { s_sum[warp] = S; s_sum[kTopmThreads / 32 + warp] = T; }
  __syncthreads();
  if (tid == 0) {
    double St = 0.0, Tt = 0.0;
    for (int w = 0; w < kTopmThreads / 32; ++w) { St += s_sum[w]; Tt += s_sum[kTopmThreads / 32 + w]; }
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

// The rows that still need their sums (active, and not served by the candidates of the expand pass): row i of the
// [B, F] grid belongs to CTA i mod gridDim.x, which finds its rows first and then takes them one after the other.
template <bool BF16>
__global__ void __launch_bounds__(kTopmThreads) topm_entropy_kernel(const void *logits, long long seq_stride,
                                                                    long long row_stride, int V, int M, int F, int B,
                                                                    const int32_t *counts, TopmAux aux, double2 *out,
                                                                    const int32_t *done) {
  extern __shared__ uint32_t s_cand[];
  __shared__ int s_list[kTopmThreads];
  __shared__ int s_list_n;
  chain_enter();
  const long long total = (long long)B * F;
  const long long mine = total > blockIdx.x ? (total - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
  for (long long k0 = 0; k0 < mine; k0 += kTopmThreads) {
    if (threadIdx.x == 0) s_list_n = 0;
    __syncthreads();
    const long long k = k0 + threadIdx.x;
    if (k < mine) {
      const long long i = blockIdx.x + (long long)gridDim.x * k;
      const int b = (int)(i / F), j = (int)(i % F);
      int n = counts[b];
      n = n < 0 ? 0 : (n > F ? F : n);
      if (j < n && !(done && done[i])) s_list[atomicAdd(&s_list_n, 1)] = (int)i;
    }
    __syncthreads();
    const int nl = s_list_n;
    for (int q = 0; q < nl; ++q) {
      const int i = s_list[q];
      __syncthreads();                             // the previous row's shared state is no longer read
      topm_entropy_row<BF16>(logits, seq_stride, row_stride, V, M, F, aux, out, i / F, i % F, s_cand);
    }
    __syncthreads();
  }
}

// ---------------------------------------------------------------- from the candidates of the expand pass

struct TopmCollected {
  const uint4 *pool;
  const TopmSegment *seg;
  int32_t *done;
};

constexpr int kFinishThreads = 512;
constexpr int kFinishCand = 8192;      // keys of a row that fit in shared memory (several CTAs per SM)
constexpr int kFinishSegs = 64;        // segments of a row the kernel handles
constexpr int kFinishBatch = 4;        // independent 16-byte loads a thread keeps in flight
constexpr int kFinishMulti = 512;      // vectors of a row with more than one candidate that the list holds

// How many elements of a vector are at or above a floor (a floor that is an element's value, or kTopmLowestFloor).
template <bool BF16>
__device__ __forceinline__ int count_at_or_above(const uint4 &q, float floor) {
  if (BF16) {
    // the floor as a bf16 pair, rounded up if it is no bf16 value (only kTopmLowestFloor is none)
    uint32_t fb = __float_as_uint(floor);
    if (fb & 0xFFFFu) fb = (fb & 0x80000000u) ? (fb & 0xFFFF0000u) : (fb + 0x10000u) & 0xFFFF0000u;
    const uint32_t f2 = (fb >> 16) | (fb & 0xFFFF0000u);
    uint32_t g0, g1, g2, g3;                         // 0xFFFF per element at or above
    asm("set.ge.u32.bf16x2 %0, %1, %2;" : "=r"(g0) : "r"(q.x), "r"(f2));
    asm("set.ge.u32.bf16x2 %0, %1, %2;" : "=r"(g1) : "r"(q.y), "r"(f2));
    asm("set.ge.u32.bf16x2 %0, %1, %2;" : "=r"(g2) : "r"(q.z), "r"(f2));
    asm("set.ge.u32.bf16x2 %0, %1, %2;" : "=r"(g3) : "r"(q.w), "r"(f2));
    const uint32_t t = (g0 & 0x00010001u) + (g1 & 0x00010001u) + (g2 & 0x00010001u) + (g3 & 0x00010001u);
    return (int)((t & 0xFFFFu) + (t >> 16));
  }
  return (__uint_as_float(q.x) >= floor) + (__uint_as_float(q.y) >= floor) + (__uint_as_float(q.z) >= floor) +
         (__uint_as_float(q.w) >= floor);
}

// One CTA per active row: the elements at or above the row's highest collection floor, out of the values that the
// expand pass set aside, and Eq. 3's sums from them if there are at least M (then the M largest are among them).
template <bool BF16>
__global__ void __launch_bounds__(kFinishThreads) topm_finish_kernel(int M, int F, const int32_t *counts, TopmAux aux,
                                                                     TopmCollected col, double2 *out) {
  extern __shared__ uint32_t s_cand[];
  __shared__ double s_sum[2 * (kFinishThreads / 32)];
  __shared__ unsigned s_need, s_count, s_multi_n;
  __shared__ uint4 s_multi[kFinishMulti];
  __shared__ int s_first[kFinishSegs], s_start[kFinishSegs + 1];
  __shared__ unsigned long long s_top;
  __shared__ float s_floor;
  __shared__ int s_ok;
  const int b = blockIdx.y, j = blockIdx.x, tid = threadIdx.x, lane = tid & 31;
  chain_enter();
  int n = counts[b];
  n = n < 0 ? 0 : (n > F ? F : n);
  if (j >= n) return;
  const PassInfo info = *aux.info;
  const int a = aux.row_off[b] + j;
  const long long first_vec = (long long)a * (info.vec_per_row + info.pad) + info.pad;
  const int c_first = (int)(first_vec / info.span);
  int n_splits = (int)((first_vec + info.vec_per_row - 1) / info.span) - c_first + 1;
  if (n_splits > aux.max_splits) n_splits = aux.max_splits;
  // ---- the row's segments: warp 0, two per lane
  if (tid < 32) {
    unsigned long long top = 0ull;
    float floor = kTopmLowestFloor;
    bool ok = n_splits <= kFinishSegs;
    int cnt[2] = {0, 0};
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int sp = lane * 2 + h;
      if (sp < n_splits && sp < kFinishSegs) {
        const size_t slot = (size_t)a * aux.max_splits + sp;
        const unsigned long long k = aux.part_held[slot];
        top = k > top ? k : top;
        const TopmSegment rec = col.seg[slot];
        ok = ok && rec.n >= 0;
        floor = fmaxf(floor, rec.floor);
        cnt[h] = rec.n > 0 ? rec.n : 0;
        s_first[sp] = rec.first;
      }
    }
    int inc = cnt[0] + cnt[1];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(kFull, inc, o);
      if (lane >= o) inc += v;
    }
    if (lane * 2 < kFinishSegs) {
      s_start[lane * 2 + 1] = inc - cnt[1];
      s_start[lane * 2 + 2] = inc;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const unsigned long long t2 = __shfl_xor_sync(kFull, top, o);
      top = t2 > top ? t2 : top;
      floor = fmaxf(floor, __shfl_xor_sync(kFull, floor, o));
    }
    ok = __all_sync(kFull, ok);
    if (lane == 0) { s_start[0] = 0; s_top = top; s_floor = floor; s_ok = ok; s_count = 0u; s_multi_n = 0u; }
  }
  __syncthreads();
  const float mf = key_value(s_top);
  const float floor = s_floor;
  const int n_seg = n_splits < kFinishSegs ? n_splits : kFinishSegs;
  const int total = s_start[n_seg];
  if (s_ok && s_top != 0ull && mf < INFINITY) {      // (uniform)
    // A thread takes a vector at a time.  Nearly every vector holds exactly one element at or above the floor, and
    // that element is the vector's maximum: two packed operations per word give the count and the maximum without
    // taking the vector apart, and a vote closes the maxima up.  The few vectors with more go to a list first and
    // are taken apart afterwards, one element per thread.
    using VT = Vec<BF16>;
    const uint32_t lo = BF16 ? kLowestBf16x2 : __float_as_uint(kLowestF32);
    const unsigned lt_mask = (1u << lane) - 1u;
    int sp = 0;
    for (int v0 = 0; v0 < total; v0 += kFinishThreads * kFinishBatch) {
      uint4 q[kFinishBatch];
#pragma unroll
      for (int k = 0; k < kFinishBatch; ++k) {
        const int v = v0 + k * kFinishThreads + tid;
        q[k] = make_uint4(lo, lo, lo, lo);
        if (v < total) {
          while (v >= s_start[sp + 1]) ++sp;         // (v rises, so does its segment)
          q[k] = col.pool[(long long)s_first[sp] + (v - s_start[sp])];
        }
      }
      unsigned m1[kFinishBatch], m2[kFinishBatch], n1 = 0u, n2 = 0u;       // (the counts are the same in every lane)
#pragma unroll
      for (int k = 0; k < kFinishBatch; ++k) {
        const int c = count_at_or_above<BF16>(q[k], floor);
        m1[k] = __ballot_sync(kFull, c == 1);
        m2[k] = __ballot_sync(kFull, c > 1);
        n1 += __popc(m1[k]);
        n2 += __popc(m2[k]);
      }
      unsigned base1 = 0u, base2 = 0u;
      if (lane == 0) {
        if (n1) base1 = atomicAdd(&s_count, n1);
        if (n2) base2 = atomicAdd(&s_multi_n, n2);
      }
      base1 = __shfl_sync(kFull, base1, 0);
      base2 = __shfl_sync(kFull, base2, 0);
#pragma unroll
      for (int k = 0; k < kFinishBatch; ++k) {
        if ((m1[k] >> lane) & 1u) {
          const unsigned pos = base1 + __popc(m1[k] & lt_mask);
          if (pos < (unsigned)kFinishCand) s_cand[pos] = f32_orderable(__float_as_uint(VT::vmax(q[k])));
        }
        if ((m2[k] >> lane) & 1u) {
          const unsigned pos = base2 + __popc(m2[k] & lt_mask);
          if (pos < (unsigned)kFinishMulti) s_multi[pos] = q[k];
        }
        base1 += __popc(m1[k]);
        base2 += __popc(m2[k]);
      }
    }
    __syncthreads();
    const unsigned n_multi = s_multi_n;
    if (n_multi <= (unsigned)kFinishMulti) {         // (uniform; else too many for the list: the row is read again)
      const unsigned n_el = n_multi * VT::N;
      for (unsigned e0 = 0; e0 < n_el; e0 += kFinishThreads) {
        const unsigned e = e0 + tid;
        float x = -INFINITY;
        if (e < n_el) {
          if (BF16) x = __uint_as_float((uint32_t)reinterpret_cast<const uint16_t *>(s_multi)[e] << 16);
          else x = reinterpret_cast<const float *>(s_multi)[e];
        }
        const unsigned mm = __ballot_sync(kFull, x >= floor);
        unsigned base = 0u;
        if (lane == 0 && mm) base = atomicAdd(&s_count, __popc(mm));
        base = __shfl_sync(kFull, base, 0);
        const unsigned pos = base + __popc(mm & lt_mask);
        if (x >= floor && pos < (unsigned)kFinishCand) s_cand[pos] = f32_orderable(__float_as_uint(x));
      }
    }
    __syncthreads();
    const unsigned n_c = s_count;
    if (n_multi <= (unsigned)kFinishMulti && n_c >= (unsigned)M && n_c <= (unsigned)kFinishCand) {
      select_and_sum<BF16, kFinishThreads>(s_cand, n_c, M, mf, f32_orderable(__float_as_uint(floor)), (uint32_t)(s_top >> 32),
                                           s_sum, &s_need, &out[(size_t)b * F + j]);
      if (tid == 0) col.done[(size_t)b * F + j] = 1;
      return;
    }
  }
  if (tid == 0) col.done[(size_t)b * F + j] = 0;
}

}  // namespace

static size_t topm_dynamic_smem() { return (size_t)kTopmCand * sizeof(uint32_t); }

cudaError_t prepare_topm_pass() {
  const int bytes = (int)topm_dynamic_smem();
  cudaError_t e = cudaFuncSetAttribute(topm_entropy_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(topm_entropy_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  const int fin = kFinishCand * (int)sizeof(uint32_t);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(topm_finish_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, fin);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(topm_finish_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, fin);
  return e;
}

cudaError_t launch_topm_entropy(const void *logits, int64_t seq_stride, int64_t row_stride, int V, int M, int F,
                                int B, const int32_t *counts, const TreeState &t, double2 *out, const int32_t *done,
                                int n_ctas, int dtype, cudaStream_t s) {
  const long long rows = (long long)B * F;
  const dim3 grid((unsigned)(rows < n_ctas ? rows : n_ctas));     // a CTA fills an SM
  TopmAux aux;
  aux.part_held = t.part_held; aux.info = t.info_draft; aux.row_off = t.row_off_draft; aux.max_splits = t.max_splits;
  const size_t smem = topm_dynamic_smem();
  if (dtype == C2T_BF16)
    return launch_chained(topm_entropy_kernel<true>, grid, dim3(kTopmThreads), smem, s, logits, seq_stride, row_stride, V, M, F,
                          B, counts, aux, out, done);
  return launch_chained(topm_entropy_kernel<false>, grid, dim3(kTopmThreads), smem, s, logits, seq_stride, row_stride, V, M, F,
                        B, counts, aux, out, done);
}

cudaError_t launch_topm_finish(int M, int F, int B, const int32_t *counts, const TreeState &t, double2 *out, int dtype,
                               cudaStream_t s) {
  const dim3 grid(F, B);
  TopmAux aux;
  aux.part_held = t.part_held; aux.info = t.info_draft; aux.row_off = t.row_off_draft; aux.max_splits = t.max_splits;
  TopmCollected col;
  col.pool = t.topm_pool; col.seg = t.topm_seg; col.done = t.topm_done;
  const size_t smem = (size_t)kFinishCand * sizeof(uint32_t);
  if (dtype == C2T_BF16)
    return launch_chained(topm_finish_kernel<true>, grid, dim3(kFinishThreads), smem, s, M, F, counts, aux, col, out);
  return launch_chained(topm_finish_kernel<false>, grid, dim3(kFinishThreads), smem, s, M, F, counts, aux, col, out);
}

}  // namespace c2t
