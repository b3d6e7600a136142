// The expand pass: one streaming read of every active draft-logits row, giving per row the
// softmax normaliser and entropy sums and the K largest logits (ties to the lower token id)
//                                                        (Sec. 4.2.1, Eq. 2, Sec. 4.2.2).
//
// Work partition.  The active rows (a device-side count per sequence) are laid end to end as
// n_rows * vec_per_row 16-byte vectors and cut into equal contiguous spans, one per CTA of a
// persistent grid (three CTAs of 256 threads per SM), so every CTA streams the same number of
// bytes whatever the row count.  A span may cover the tail of one row, some whole rows and the
// head of another; each (row, CTA) piece is a "segment" and produces one partial record.  The
// pruning kernel merges the partials of a row in double precision.
//
// Data movement.  A thread works on groups of four 16-byte vectors, 256 vectors apart.  Each
// thread owns 4 x 16 bytes in each of two shared-memory slots and fills them with cp.async:
// while group n is in registers, groups n+1 and n+2 are in flight, across segment boundaries
// too.  A thread reads back only what it copied itself, so the only wait is on its own copies
// (cp.async.wait_group); nothing waits on another thread's progress except at __syncthreads,
// of which a segment boundary has two.
//
// Sums.  In base-2 units relative to a warp-uniform offset c = -m log2(e):  t = x log2(e) + c,
// S = sum 2^t, U = sum 2^t t  (one unpack, FMA, ex2, add, FMA per element).  They cover all
// elements of the segment except one per warp: each warp holds its running maximum out of the
// sums and hands it on as an exact (value, token) key, releasing the previous one into the
// sums when a larger element arrives.  The row maximum is therefore never added in fp32, so
// the sums keep fp32 relative accuracy with respect to "everything but the maximum" however
// peaked the row is; the merge adds the held keys in double precision.  Which element is held
// depends only on the warp's own data and all reductions run in a fixed order, so the sums are
// reproducible bit for bit.  m stays within 60 of every summed value.  (x log2(e) uses the
// fp32 constant: a relative error of 1.3e-8 |x| in an element's weight, far inside tolerance.)
//
// Top-K.  Finding the K largest has no effect on the sums.  A shared list of the K largest
// VALUES seen (32-bit atomicMax cascade) gives the filter; every element at or above the
// filter when it is read appends its key to a buffer, from which one warp selects the K
// largest keys at the end of the segment.  The first group seeds the filter with the K-th
// largest lane maximum.  A buffer overflow (e.g. a row sorted ascending) falls back to K exact
// arg-max rescans of the segment.
//
// The two rare paths (a lane met the filter; a warp met a new maximum) are out-of-line
// functions that take and return everything BY VALUE: a hot variable whose address escaped
// into a call would live in local memory for the whole kernel.
#include "vocab_common.cuh"

namespace c2t {
namespace {

constexpr int NT = kExpandThreads;
constexpr int kEWarps = NT / 32;
constexpr int kBufCap = 256;       // top-K candidate keys a segment can collect before the exact fallback

// ---------------------------------------------------------------- sums

struct Acc {
  float S0, S1, U0, U1;
};

__device__ __forceinline__ void acc_clear(Acc &a) { a.S0 = a.S1 = a.U0 = a.U1 = 0.f; }

// move the offset from c to new_c (the reference only rises, so new_c <= c)
__device__ __forceinline__ void acc_rescale(Acc &a, float c, float new_c) {
  const float S = a.S0 + a.S1, U = a.U0 + a.U1;
  const float d = fmaxf(new_c - c, -1e30f);          // every t shifts by d
  const float f = ex2f(d);
  a.S0 = S * f;
  a.U0 = f * (U + d * S);
  a.S1 = a.U1 = 0.f;
}

__device__ __forceinline__ void acc_scalar(Acc &a, float c, float x) {
  const float t = fmaf(x, kLog2e, c);
  const float e = ex2f(t);
  a.S0 += e;
  a.U0 = fmaf(e, t, a.U0);
}

template <bool BF16>
__device__ __forceinline__ void acc_vector(Acc &a, const uint4 &q, float c) {
  float x[Vec<BF16>::N];
  Vec<BF16>::unpack(q, x);
#pragma unroll
  for (int i = 0; i < Vec<BF16>::N; i += 2) {
    const float t0 = fmaf(x[i], kLog2e, c), t1 = fmaf(x[i + 1], kLog2e, c);
    const float e0 = ex2f(t0), e1 = ex2f(t1);
    a.S0 += e0;
    a.S1 += e1;
    a.U0 = fmaf(e0, t0, a.U0);
    a.U1 = fmaf(e1, t1, a.U1);
  }
}

// (c, S, U) of two disjoint sets -> their union, relative to the smaller offset (larger reference)
__device__ __forceinline__ void combine(float &c, float &S, float &U, float c2, float S2, float U2) {
  const float C = fminf(c, c2);
  const float d1 = fmaxf(C - c, -1e30f), d2 = fmaxf(C - c2, -1e30f);
  const float f1 = ex2f(d1), f2 = ex2f(d2);
  U = f1 * (U + d1 * S) + f2 * (U2 + d2 * S2);
  S = f1 * S + f2 * S2;
  c = C;
}

// element i of a vector := -2^127 (adds exactly 0 to the sums)
template <bool BF16>
__device__ __forceinline__ void mask_element(uint4 &q, int i) {
  uint32_t *w = reinterpret_cast<uint32_t *>(&q);
  if (BF16) {
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (i == 2 * k) w[k] = (w[k] & 0xFFFF0000u) | 0x0000FF00u;
      if (i == 2 * k + 1) w[k] = (w[k] & 0x0000FFFFu) | 0xFF000000u;
    }
  } else {
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if (i == k) w[k] = __float_as_uint(kLowestF32);
  }
}

// ---------------------------------------------------------------- segment state

// Shared by the CTA for the segment being streamed.
struct SegShared {
  unsigned long long buf[kBufCap];        // keys of every element that met the filter when it was read
  unsigned long long held[kEWarps];        // per warp: the key held out of the sums
  uint32_t vals[C2T_MAX_TOPK];            // K largest values seen (orderable form); vals[K-1] is the filter
  uint32_t warm[kEWarps * C2T_MAX_TOPK];
  float red[kEWarps][3];
  float m0;
  int cnt;
  int overflow;
};

// Per thread.
struct SegState {
  Acc acc;
  float m, c, mw, thr;      // reference, offset -m log2(e), warp's running maximum, top-K filter
  unsigned long long held;  // warp-uniform
};

struct Group {
  uint4 q[4];
};

// An element at or above the filter: remember its key, and raise the filter if its value is new.
__device__ __forceinline__ void push_candidate(SegShared &sh, int K, float x, uint32_t tok, float thr) {
  const int pos = atomicAdd(&sh.cnt, 1);
  if (pos < kBufCap) sh.buf[pos] = make_key(x, tok);
  else sh.overflow = 1;
  if (x > thr) {
    const uint32_t floor_u = f32_orderable(__float_as_uint(thr));
    uint32_t carry = f32_orderable(__float_as_uint(x));
    for (int s = 0; s < K; ++s) {
      const uint32_t old = atomicMax(&sh.vals[s], carry);
      if (old < carry) carry = old;
      if (carry <= floor_u) break;
    }
  }
}

template <bool BF16>
__device__ __forceinline__ void lane_event(SegShared &sh, int K, const uint4 &q, uint32_t tok0, float thr) {
  float x[Vec<BF16>::N];
  Vec<BF16>::unpack(q, x);
#pragma unroll 1
  for (int i = 0; i < Vec<BF16>::N; ++i)
    if (x[i] >= thr) push_candidate(sh, K, x[i], tok0 + i, thr);
}

// Rare, lane-divergent, out of line: some vector of this thread's group holds an element at or
// above the filter.  No effect on the sums.
template <bool BF16>
__device__ __noinline__ void group_filter_events(SegShared *sh, int K, Group g, int vt, int v1, float thr) {
  using VT = Vec<BF16>;
#pragma unroll 1
  for (int u = 0; u < 4; ++u) {
    const int v = vt + u * NT;
    if (v < v1 && VT::vmax(g.q[u]) >= thr) lane_event<BF16>(*sh, K, g.q[u], (uint32_t)v * VT::N, thr);
  }
}

// Rare, warp-uniform, out of line: some lane of the warp read an element above the warp's
// running maximum.  Does everything for this group (filter events, hold-out, sums) and returns
// the thread's new state.
template <bool BF16>
__device__ __noinline__ SegState group_with_new_maximum(SegShared *sh, int K, Group g, int vt, int v1, SegState st) {
  using VT = Vec<BF16>;
  const int lane = threadIdx.x & 31;
#pragma unroll 1
  for (int u = 0; u < 4; ++u) {
    const int v = vt + u * NT;
    const bool valid = v < v1;
    uint4 q = g.q[u];
    const float vm = VT::vmax(q);
    if (valid && vm >= st.thr) lane_event<BF16>(*sh, K, q, (uint32_t)v * VT::N, st.thr);   // before any masking
    const bool rec = valid && vm > st.mw;
    if (__any_sync(kFull, rec)) {
      // the warp's new maximum is held out (as an exact key); the previous one joins lane 0's sums
      unsigned long long mine = 0ull;
      int idx = 0;
      if (rec) {
        float x[VT::N];
        VT::unpack(q, x);
#pragma unroll
        for (int i = VT::N - 1; i >= 0; --i)
          if (x[i] == vm) idx = i;
        mine = make_key(vm, (uint32_t)v * VT::N + idx);
      }
      unsigned long long best = mine;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long other = __shfl_xor_sync(kFull, best, o);
        best = other > best ? other : best;
      }
      const float new_mw = key_value(best);
      if (new_mw - st.m > 60.f) {          // keep every summed element within e^60 of the reference
        const float new_c = -new_mw * kLog2e;
        acc_rescale(st.acc, st.c, new_c);
        st.m = new_mw;
        st.c = new_c;
      }
      if (lane == 0 && st.held != 0ull) acc_scalar(st.acc, st.c, key_value(st.held));
      if (rec && mine == best) mask_element<BF16>(q, idx);
      st.held = best;
      st.mw = new_mw;
    }
    acc_vector<BF16>(st.acc, q, st.c);     // vectors past the segment hold -2^127: they add 0
  }
  return st;
}

// ---------------------------------------------------------------- segments of a span

struct Segment {
  const char *row;
  int a, v0, v1;     // vectors [v0, v1) of active row a
};

struct SegWalk {
  int a, v0, left, vec_per_row;
  __device__ SegWalk(const Partition &pt) : vec_per_row(pt.vec_per_row) {
    a = (int)(pt.start / pt.vec_per_row);
    v0 = (int)(pt.start - (long long)a * pt.vec_per_row);
    left = (int)(pt.end - pt.start);
  }
  __device__ bool done() const { return left <= 0; }
  __device__ Segment take(const PassParams &p, const int *s_off, size_t esz) {
    Segment g;
    const int room = vec_per_row - v0;
    const int n = left < room ? left : room;
    g.a = a; g.v0 = v0; g.v1 = v0 + n;
    const int b = find_sequence(s_off, p.B, a);
    const int j = a - s_off[b];
    g.row = reinterpret_cast<const char *>(p.logits) + ((size_t)b * p.seq_stride + (size_t)j * p.row_stride) * esz;
    left -= n;
    ++a;
    v0 = 0;
    return g;
  }
};

// ---------------------------------------------------------------- asynchronous prefetch ring
//
// Every thread owns 4 x 16 bytes in each of the two slots of a shared-memory ring and fills
// them with cp.async (global -> shared, no registers held): while group n is being worked on,
// groups n+1 and n+2 are in flight.  A thread only ever reads back what it copied itself, so
// the only wait is cp.async.wait_group on its own copies; no barrier is involved and the
// prefetch runs ahead across segment boundaries.

__device__ __forceinline__ void cp_async_16(void *smem_dst, const void *gmem_src) {
  const uint32_t dst = (uint32_t)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// The groups of a span in order: group = four vectors per thread, NT apart, of one segment.
struct GroupCursor {
  SegWalk walk;
  Segment seg;     // the segment the current group belongs to
  int tv0;         // first vector of the current group (CTA-uniform); the thread's are tv0+tid+u*NT
  bool valid;
  __device__ GroupCursor(const Partition &pt, const PassParams &p, const int *s_off, size_t esz) : walk(pt) {
    seg = walk.take(p, s_off, esz);
    tv0 = seg.v0;
    valid = true;
  }
  __device__ bool last_of_segment() const { return tv0 + 4 * NT >= seg.v1; }
  __device__ void advance(const PassParams &p, const int *s_off, size_t esz) {
    tv0 += 4 * NT;
    if (tv0 >= seg.v1) {
      if (walk.done()) { valid = false; return; }
      seg = walk.take(p, s_off, esz);
      tv0 = seg.v0;
    }
  }
};

// Requests the whole vectors of the cursor's group into the thread's places of a ring slot.
__device__ __forceinline__ void prefetch_group(const GroupCursor &c, uint4 *slot, int v_full) {
  if (c.valid) {
    const int lim = c.seg.v1 < v_full ? c.seg.v1 : v_full;
    const uint4 *src = reinterpret_cast<const uint4 *>(c.seg.row) + c.tv0 + (int)threadIdx.x;
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (c.tv0 + (int)threadIdx.x + u * NT < lim) cp_async_16(slot + threadIdx.x + u * NT, src + u * NT);
  }
  cp_async_commit();
}

// Takes the cursor's group out of a ring slot (its copies have completed) into registers and
// clamps it.  Vectors past the segment end become -2^127, which adds exactly 0 to the sums; a
// ragged last vector of a row is assembled from scalar loads.
template <bool BF16>
__device__ __forceinline__ void take_group(Group &g, const GroupCursor &c, const uint4 *slot, int v_full, int V) {
  using VT = Vec<BF16>;
  const uint32_t lo = BF16 ? kLowestBf16x2 : __float_as_uint(kLowestF32);
  const int vt = c.tv0 + (int)threadIdx.x;
  if (__all_sync(kFull, vt + 3 * NT < (c.seg.v1 < v_full ? c.seg.v1 : v_full))) {
#pragma unroll
    for (int u = 0; u < 4; ++u) g.q[u] = slot[threadIdx.x + u * NT];
  } else {
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int v = vt + u * NT;
      g.q[u] = make_uint4(lo, lo, lo, lo);
      if (v < c.seg.v1) g.q[u] = v < v_full ? slot[threadIdx.x + u * NT] : VT::load(c.seg.row, v, v_full, V);
    }
  }
#pragma unroll
  for (int u = 0; u < 4; ++u) VT::clamp(g.q[u]);
}

// Exact fallback for a segment whose candidate buffer overflowed: K rounds of a CTA-wide
// arg-max over the segment, each round below the key found by the round before.
template <bool BF16>
__device__ __noinline__ void select_by_rescan(int K, int V, int v_full, const char *row, int v0, int v1,
                                              unsigned long long *out_keys, unsigned long long *s_scratch) {
  using VT = Vec<BF16>;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  unsigned long long bound = ~0ull;
  for (int r = 0; r < K; ++r) {
    unsigned long long best = 0ull;
    for (int v = v0 + tid; v < v1; v += NT) {
      uint4 q = VT::load(row, v, v_full, V);
      VT::clamp(q);
      float x[VT::N];
      VT::unpack(q, x);
#pragma unroll
      for (int i = 0; i < VT::N; ++i) {
        if (x[i] != x[i]) continue;
        const unsigned long long key = make_key(x[i], (uint32_t)v * VT::N + i);
        if (key < bound && key > best) best = key;
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const unsigned long long other = __shfl_xor_sync(kFull, best, o);
      best = other > best ? other : best;
    }
    __syncthreads();
    if (lane == 0) s_scratch[warp] = best;
    __syncthreads();
    best = 0ull;
    for (int w = 0; w < kEWarps; ++w) best = s_scratch[w] > best ? s_scratch[w] : best;
    if (tid == 0) out_keys[r] = best;
    bound = best;
  }
}

// Warm-up, stage 1 (every warp, no barrier): the warp's K largest lane maxima of a segment's
// first group, descending, into shared memory.
template <bool BF16>
__device__ __forceinline__ void warmup_stage1(SegShared &sh, int K, const Group &g, int vt, int v1) {
  using VT = Vec<BF16>;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float lmax = -INFINITY;
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    if (vt + u * NT < v1) {
      const float vm = VT::vmax(g.q[u]);
      if (vm == vm) lmax = fmaxf(lmax, vm);
    }
  }
  uint32_t live = f32_orderable(__float_as_uint(lmax)), mine = 0;
  for (int r = 0; r < K; ++r) {
    const uint32_t mx = __reduce_max_sync(kFull, live);
    const unsigned bal = __ballot_sync(kFull, live == mx);
    if (lane == __ffs(bal) - 1) live = 0;
    if (lane == r) mine = mx;
  }
  if (lane < K) sh.warm[warp * K + lane] = mine;
}

// Warm-up, stage 2 (warp 0, between two barriers): the K-th largest of the union of the sorted
// per-warp lists seeds the filter (a valid lower bound of the segment's K-th largest element),
// their maximum becomes the reference of the sums; the candidate buffer is emptied.
__device__ __forceinline__ void warmup_stage2(SegShared &sh, int K) {
  const int lane = threadIdx.x & 31;
  int head = 0;
  uint32_t mx = 0, first = 0;
  for (int r = 0; r < K; ++r) {   // lane w walks list w
    const uint32_t h = (lane < kEWarps && head < K) ? sh.warm[lane * K + head] : 0u;
    mx = __reduce_max_sync(kFull, h);
    if (r == 0) first = mx;
    const unsigned bal = __ballot_sync(kFull, h == mx);
    if (lane == __ffs(bal) - 1) ++head;
  }
  if (lane < K) sh.vals[lane] = mx;
  if (lane == 0) {
    sh.m0 = __uint_as_float(f32_from_orderable(first));
    sh.cnt = 0;
    sh.overflow = 0;
  }
}

__device__ __forceinline__ void state_init(const SegShared &sh, SegState &st) {
  acc_clear(st.acc);
  st.m = sh.m0;                                      // warp-uniform reference of the sums
  st.c = -st.m * kLog2e;
  st.mw = __uint_as_float(f32_from_orderable(f32_orderable(__float_as_uint(st.m)) - 1u));   // just below m0
  st.held = 0ull;
}

// End of a segment, every warp, before the barrier: the warp's sums (fixed order) and held key.
__device__ __forceinline__ void publish_warp_sums(SegShared &sh, const SegState &st) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float S = st.acc.S0 + st.acc.S1, U = st.acc.U0 + st.acc.U1;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {                   // the offset is warp-uniform: plain sums
    S += __shfl_down_sync(kFull, S, o);
    U += __shfl_down_sync(kFull, U, o);
  }
  if (lane == 0) {
    sh.red[warp][0] = st.c; sh.red[warp][1] = S; sh.red[warp][2] = U;
    sh.held[warp] = st.held;
  }
}

// End of a segment, warp 0, after the barrier: merge the warps' sums and emit the partial record.
__device__ __forceinline__ void emit_partial(SegShared &sh, const PassParams &p, size_t slot, bool overflow) {
  const int lane = threadIdx.x & 31;
  const int K = p.K;
  float cc = lane < kEWarps ? sh.red[lane][0] : sh.red[0][0];
  float S = lane < kEWarps ? sh.red[lane][1] : 0.f;
  float U = lane < kEWarps ? sh.red[lane][2] : 0.f;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float c_o = __shfl_down_sync(kFull, cc, o);
    const float S_o = __shfl_down_sync(kFull, S, o);
    const float U_o = __shfl_down_sync(kFull, U, o);
    combine(cc, S, U, c_o, S_o, U_o);
  }
  if (lane < kEWarps) p.part_held[slot * kEWarps + lane] = sh.held[lane];
  int n_keys = K;
  if (!overflow) {
    // the K largest keys of the buffer, sorted, by counting
    const int n = sh.cnt < kBufCap ? sh.cnt : kBufCap;
    n_keys = n < K ? n : K;
    if (n <= 32) {                                      // one key per lane, ranked through shuffles
      const unsigned long long key = lane < n ? sh.buf[lane] : 0ull;
      int rank = 0;
      for (int r = 0; r < n; ++r) rank += __shfl_sync(kFull, key, r) > key;
      if (lane < n && rank < K) p.part_keys[slot * K + rank] = key;
    } else {
      for (int i = lane; i < n; i += 32) {
        const unsigned long long key = sh.buf[i];
        int rank = 0;
        for (int r = 0; r < n; ++r) rank += sh.buf[r] > key;
        if (rank < K) p.part_keys[slot * K + rank] = key;
      }
    }
    for (int r = n_keys + lane; r < K; r += 32) p.part_keys[slot * K + r] = 0ull;
  }
  if (lane == 0) p.part_stats[slot] = make_float4(cc, S, U, __int_as_float(n_keys));
}

template <bool BF16>
__global__ void __launch_bounds__(kExpandThreads, kExpandCtasPerSm) expand_pass_kernel(PassParams p) {
  using VT = Vec<BF16>;
  extern __shared__ __align__(16) unsigned char s_dyn[];     // ring: 2 slots of 4*NT vectors, then row offsets
  __shared__ SegShared sh;
  uint4 *ring = reinterpret_cast<uint4 *>(s_dyn);
  int *s_off = reinterpret_cast<int *>(s_dyn + 2 * 4 * NT * sizeof(uint4));

  const int K = p.K;
  const int warp = threadIdx.x >> 5;
  const int n_rows = build_row_offsets(p.counts, p.B, p.rows_per_seq_max, s_off);
  const Partition pt = make_partition<VT::N>(p, n_rows);
  if (pt.start >= pt.end) return;

  const size_t esz = BF16 ? 2 : 4;
  GroupCursor cur(pt, p, s_off, esz);      // the group being worked on
  GroupCursor pre = cur;                   // the group being requested, two ahead
  prefetch_group(pre, ring, pt.v_full);
  pre.advance(p, s_off, esz);
  prefetch_group(pre, ring + 4 * NT, pt.v_full);
  pre.advance(p, s_off, esz);
  unsigned n = 0;                          // index of the current group: its ring slot is n & 1

  Group g;
  cp_async_wait<1>();
  take_group<BF16>(g, cur, ring, pt.v_full, p.V);
  prefetch_group(pre, ring, pt.v_full);
  pre.advance(p, s_off, esz);
  warmup_stage1<BF16>(sh, K, g, cur.tv0 + (int)threadIdx.x, cur.seg.v1);
  __syncthreads();
  if (warp == 0) warmup_stage2(sh, K);
  __syncthreads();

  for (;;) {
    // ---- one segment; its first group is in registers and the filter is seeded
    const Segment seg = cur.seg;
    SegState st;
    state_init(sh, st);
    for (;;) {
      const int vt = cur.tv0 + (int)threadIdx.x;
      st.thr = __uint_as_float(f32_from_orderable(*reinterpret_cast<volatile uint32_t *>(&sh.vals[K - 1])));
      const float vm4 = fmaxf(fmaxf(VT::vmax(g.q[0]), VT::vmax(g.q[1])), fmaxf(VT::vmax(g.q[2]), VT::vmax(g.q[3])));
      if (__any_sync(kFull, vm4 > st.mw && vt < seg.v1)) {
        st = group_with_new_maximum<BF16>(&sh, K, g, vt, seg.v1, st);
      } else {
        if (vm4 >= st.thr && vt < seg.v1) group_filter_events<BF16>(&sh, K, g, vt, seg.v1, st.thr);
#pragma unroll
        for (int u = 0; u < 4; ++u) acc_vector<BF16>(st.acc, g.q[u], st.c);
      }
      const bool last = cur.last_of_segment();
      cur.advance(p, s_off, esz);
      ++n;
      if (cur.valid) {                       // next group (of this or of the next segment) into registers
        cp_async_wait<1>();
        uint4 *slot = ring + (n & 1u) * 4 * NT;
        take_group<BF16>(g, cur, slot, pt.v_full, p.V);
        prefetch_group(pre, slot, pt.v_full);
        pre.advance(p, s_off, esz);
      }
      if (last) break;
    }
    // ---- segment boundary: two barriers; warp 0 closes this segment and seeds the next
    publish_warp_sums(sh, st);
    const bool more = cur.valid;
    if (more) warmup_stage1<BF16>(sh, K, g, cur.tv0 + (int)threadIdx.x, cur.seg.v1);
    __syncthreads();
    const bool overflow = sh.overflow != 0;
    const int split = blockIdx.x - (int)(((long long)seg.a * pt.vec_per_row) / pt.span);
    const size_t slot_id = (size_t)seg.a * p.max_splits + split;
    if (warp == 0) emit_partial(sh, p, slot_id, overflow);
    if (overflow)
      select_by_rescan<BF16>(K, p.V, pt.v_full, seg.row, seg.v0, seg.v1, p.part_keys + slot_id * K, sh.held);
    if (warp == 0 && more) warmup_stage2(sh, K);
    __syncthreads();
    if (!more) break;
  }
  cp_async_wait<0>();
}

}  // namespace

int max_splits_for(int vocab, int elem_bytes, int grid) {
  const int vec = 16 / elem_bytes;
  const int vec_per_row = (vocab + vec - 1) / vec;
  int by_span = (vec_per_row + kMinSpanVectors - 1) / kMinSpanVectors;
  if (by_span > grid) by_span = grid;
  return by_span + 1;
}

static size_t expand_dynamic_smem(int B) {
  return 2 * 4 * (size_t)kExpandThreads * sizeof(uint4) + ((size_t)B + 1) * sizeof(int);
}

cudaError_t prepare_expand_pass() {
  const int bytes = (int)expand_dynamic_smem(C2T_MAX_BATCH);
  cudaError_t e = cudaFuncSetAttribute(expand_pass_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(expand_pass_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
}

cudaError_t launch_expand_pass(const PassParams &p, int dtype, int grid, cudaStream_t s) {
  const size_t smem = expand_dynamic_smem(p.B);
  if (dtype == C2T_BF16) expand_pass_kernel<true><<<grid, kExpandThreads, smem, s>>>(p);
  else expand_pass_kernel<false><<<grid, kExpandThreads, smem, s>>>(p);
  return cudaGetLastError();
}

}  // namespace c2t
