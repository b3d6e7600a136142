// The arg-max pass over target logits: per active row the largest logit, ties to the lower
// token id, for the greedy acceptance walk (Sec. 5 Metrics).  Same even partition of the
// active rows as the expand pass; plain 128-bit loads, four in flight per thread.
#include "vocab_common.cuh"

namespace c2t {
namespace {

// ---------------------------------------------------------------- argmax ----

template <bool BF16>
__global__ void __launch_bounds__(kPassThreads, kPassCtasPerSm) argmax_pass_kernel(PassParams p) {
  using VT = Vec<BF16>;
  __shared__ int s_off[C2T_MAX_BATCH + 1];
  __shared__ unsigned long long s_best[kWarps];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  chain_enter();
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
    const int j = p.row_sel ? p.row_sel[b] : a - s_off[b];
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
      if (lane == 0 && C2T_IN_BOUNDS(slot, p.n_slots, p.status)) p.part_best[slot] = best;
    }
    __syncthreads();
    pos += seg;
    ++a;
    v0 = 0;
  }
}

}  // namespace

cudaError_t launch_argmax_pass(const PassParams &p, int dtype, int grid, cudaStream_t s) {
  if (dtype == C2T_BF16) return launch_chained(argmax_pass_kernel<true>, dim3(grid), dim3(kPassThreads), 0, s, p);
  return launch_chained(argmax_pass_kernel<false>, dim3(grid), dim3(kPassThreads), 0, s, p);
}

}  // namespace c2t
