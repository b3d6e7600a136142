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

// ---------------------------------------------------------------- segment state

constexpr int kDefer = 6;          // vectors a thread can set aside per segment

// Shared by the CTA for the segment being streamed.
struct SegShared {
  unsigned long long buf[kBufCap];        // keys of all elements at or above the filter
  unsigned long long held[kEWarps];       // per warp: the key held out of the sums
  float red[kEWarps][3];                  // per warp: offset c, S, U
  uint32_t warm[kEWarps * C2T_MAX_TOPK];
  float thr0;                             // the filter of this segment, fixed once seeded
  float m0;                               // reference of the streamed sums (largest lane maximum of the first group)
  int cnt;                                // keys appended to buf
};

// Per thread.
struct SegState {
  Acc acc;                  // sums over the groups that stayed below the filter
  float c, thr0;            // their offset -m0 log2(e); the filter
  int n_deferred;           // vectors set aside (may exceed kDefer: then the warp redoes its share)
};

struct Group {
  uint4 q[4];
};

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

// Warm-up, stage 1 (every warp, no barrier): the warp's K largest lane maxima over the first
// two groups of a segment (the first is in registers, the second has just landed in the ring),
// descending, into shared memory.
template <bool BF16>
__device__ __forceinline__ void warmup_stage1(SegShared &sh, int K, const Group &g, int vt, int v1, int v_full,
                                              const uint4 *next_slot) {
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
  cp_async_wait<1>();                      // the group after this one (all but the newest request)
  const int lim = v1 < v_full ? v1 : v_full;
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    if (vt + (4 + u) * NT < lim) {         // same segment, whole vector: it is in the ring
      const float vm = VT::vmax(next_slot[threadIdx.x + u * NT]);
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
// per-warp lists is the segment's filter (K distinct elements are at or above it, so the K
// largest elements of the segment all are); the largest is the reference of the streamed sums.
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
  if (lane == 0) {
    sh.thr0 = __uint_as_float(f32_from_orderable(mx));
    // no data at all (every lane maximum is -inf or NaN): any finite reference will do
    sh.m0 = first == f32_orderable(0xFF800000u) ? 0.f : __uint_as_float(f32_from_orderable(first));
    sh.cnt = 0;
  }
}

// What a thread set aside while streaming: up to kDefer vectors (data and vector index), in
// its own places of shared memory, NT entries apart.
struct DeferSlots {
  uint4 *data;
  int *index;
};

// One vector that met the filter, element by element: keys at or above the filter are
// appended, everything but the held key is summed with offset cd.
template <bool BF16>
__device__ __forceinline__ void careful_vector(SegShared &sh, const uint4 &q, uint32_t tok0, float thr0,
                                               unsigned long long held, Acc &d, float cd) {
  float x[Vec<BF16>::N];
  Vec<BF16>::unpack(q, x);
#pragma unroll
  for (int i = 0; i < Vec<BF16>::N; ++i) {
    const unsigned long long key = make_key(x[i], tok0 + i);
    if (x[i] >= thr0) {
      const int pos = atomicAdd(&sh.cnt, 1);
      if (pos < kBufCap) sh.buf[pos] = key;
    }
    if (key != held) acc_scalar(d, cd, x[i]);     // (a NaN element poisons the sums, as it must)
  }
}

// the largest key of a vector (NaN elements ignored)
template <bool BF16>
__device__ __forceinline__ unsigned long long vector_best_key(const uint4 &q, uint32_t tok0) {
  float x[Vec<BF16>::N];
  Vec<BF16>::unpack(q, x);
  unsigned long long best = 0ull;
#pragma unroll
  for (int i = 0; i < Vec<BF16>::N; ++i) {
    const unsigned long long key = make_key(x[i], tok0 + i);
    if (x[i] == x[i] && key > best) best = key;
  }
  return best;
}

__device__ __forceinline__ unsigned long long warp_max_key(unsigned long long k) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const unsigned long long other = __shfl_xor_sync(kFull, k, o);
    k = other > k ? other : k;
  }
  return k;
}

// the thread's streamed sums and the sums of what it resolved become one
__device__ __forceinline__ void merge_deferred(SegState &st, bool any, float cd, const Acc &d) {
  float c = st.c, S = st.acc.S0 + st.acc.S1, U = st.acc.U0 + st.acc.U1;
  if (any) combine(c, S, U, cd, d.S0 + d.S1, d.U0 + d.U1);
  st.c = c;
  st.acc.S0 = S; st.acc.S1 = 0.f; st.acc.U0 = U; st.acc.U1 = 0.f;
}

// Fallback, per warp, for a thread that ran out of places: the warp goes over its whole share
// of the segment again, from global memory, treating every vector as set aside.
template <bool BF16>
__device__ __noinline__ unsigned long long resolve_by_rescan(SegShared *shp, const char *row, int v0t, int v1,
                                                             int v_full, int V, SegState *stp) {
  using VT = Vec<BF16>;
  SegState &st = *stp;
  acc_clear(st.acc);
  unsigned long long best = 0ull;
  for (int v = v0t; __any_sync(kFull, v < v1); v += NT) {
    if (v >= v1) continue;
    uint4 q = VT::load(row, v, v_full, V);
    VT::clamp(q);
    const unsigned long long k = vector_best_key<BF16>(q, (uint32_t)v * VT::N);
    best = k > best ? k : best;
  }
  const unsigned long long held = warp_max_key(best);
  Acc d;
  acc_clear(d);
  const float cd = -(best ? key_value(best) : 0.f) * kLog2e;
  for (int v = v0t; v < v1; v += NT) {
    uint4 q = VT::load(row, v, v_full, V);
    VT::clamp(q);
    careful_vector<BF16>(*shp, q, (uint32_t)v * VT::N, st.thr0, held, d, cd);
  }
  merge_deferred(st, best != 0ull, cd, d);
  return held;
}

// End of a segment, per warp: resolve the vectors that were set aside.  Their elements at or
// above the filter append their keys; the largest of them all is the warp's held key and stays
// out of the sums; the rest is summed relative to the thread's own largest deferred value and
// merged into the thread's streamed sums.  Uses only the warp's own data and the segment's
// filter, so the result does not depend on timing.
template <bool BF16>
__device__ __noinline__ unsigned long long resolve_deferred(SegShared *shp, DeferSlots slots, SegState *stp) {
  using VT = Vec<BF16>;
  SegState &st = *stp;
  const int n = st.n_deferred;
  unsigned long long best = 0ull;
#pragma unroll 1
  for (int i = 0; i < n; ++i) {
    const unsigned long long k = vector_best_key<BF16>(slots.data[i * NT], (uint32_t)slots.index[i * NT] * VT::N);
    best = k > best ? k : best;
  }
  const unsigned long long held = warp_max_key(best);
  Acc d;
  acc_clear(d);
  const float cd = -(best ? key_value(best) : 0.f) * kLog2e;
#pragma unroll 1
  for (int i = 0; i < n; ++i)
    careful_vector<BF16>(*shp, slots.data[i * NT], (uint32_t)slots.index[i * NT] * VT::N, st.thr0, held, d, cd);
  merge_deferred(st, best != 0ull, cd, d);
  return held;
}

// End of a segment, every warp, before the barrier: the warp's sums (fixed order) and held key.
__device__ __forceinline__ void publish_warp_sums(SegShared &sh, const SegState &st, unsigned long long held) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float c = st.c, S = st.acc.S0 + st.acc.S1, U = st.acc.U0 + st.acc.U1;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {                   // offsets may differ between lanes
    const float c_o = __shfl_down_sync(kFull, c, o);
    const float S_o = __shfl_down_sync(kFull, S, o);
    const float U_o = __shfl_down_sync(kFull, U, o);
    combine(c, S, U, c_o, S_o, U_o);
  }
  if (lane == 0) {
    sh.red[warp][0] = c; sh.red[warp][1] = S; sh.red[warp][2] = U;
    sh.held[warp] = held;
  }
}

// End of a segment, after the barrier: every thread ranks at most two of the collected keys
// (the K largest go out sorted); warp 0 merges the warps' sums and writes the record.
__device__ __forceinline__ void emit_partial(SegShared &sh, const PassParams &p, size_t slot, bool overflow) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int K = p.K;
  const int n = sh.cnt < kBufCap ? sh.cnt : kBufCap;
  if (!overflow) {
    for (int i = threadIdx.x; i < n; i += NT) {
      const unsigned long long key = sh.buf[i];
      int rank = 0;
      for (int r = 0; r < n; ++r) rank += sh.buf[r] > key;
      if (rank < K) p.part_keys[slot * K + rank] = key;
    }
    for (int r = n + threadIdx.x; r < K; r += NT) p.part_keys[slot * K + r] = 0ull;
  }
  if (warp != 0) return;
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
  if (lane == 0) p.part_stats[slot] = make_float4(cc, S, U, __int_as_float(overflow ? K : (n < K ? n : K)));
}

template <bool BF16>
__global__ void __launch_bounds__(kExpandThreads, kExpandCtasPerSm) expand_pass_kernel(PassParams p) {
  using VT = Vec<BF16>;
  // dynamic shared memory: the ring (2 slots of 4*NT vectors), the threads' deferred-group places, the row offsets
  extern __shared__ __align__(16) unsigned char s_dyn[];
  __shared__ SegShared sh;
  uint4 *ring = reinterpret_cast<uint4 *>(s_dyn);
  DeferSlots slots;
  slots.data = reinterpret_cast<uint4 *>(s_dyn + 2 * 4 * NT * sizeof(uint4)) + threadIdx.x;
  slots.index = reinterpret_cast<int *>(s_dyn + (2 * 4 + kDefer) * NT * sizeof(uint4)) + threadIdx.x;
  int *s_off = reinterpret_cast<int *>(s_dyn + (2 * 4 + kDefer) * NT * sizeof(uint4)) + kDefer * NT;

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
  warmup_stage1<BF16>(sh, K, g, cur.tv0 + (int)threadIdx.x, cur.seg.v1, pt.v_full, ring + ((n + 1) & 1u) * 4 * NT);
  __syncthreads();
  if (warp == 0) warmup_stage2(sh, K);
  __syncthreads();

  for (;;) {
    // ---- one segment; its first group is in registers and the filter is fixed
    const Segment seg = cur.seg;
    SegState st;
    acc_clear(st.acc);
    st.c = -sh.m0 * kLog2e;
    st.thr0 = sh.thr0;
    st.n_deferred = 0;
    for (;;) {
      // a vector with an element at or above the filter is set aside; the others are summed.
      // Everything summed here is below the filter, hence below the reference: no overflow.
      const int vt = cur.tv0 + (int)threadIdx.x;
      const float vm4 = fmaxf(fmaxf(VT::vmax(g.q[0]), VT::vmax(g.q[1])), fmaxf(VT::vmax(g.q[2]), VT::vmax(g.q[3])));
      if (vm4 >= st.thr0 && vt < seg.v1) {
        int v = vt;                          // rare: rolled, walking the group by rotation
#pragma unroll 1
        for (int u = 0; u < 4; ++u) {
          if (v < seg.v1 && VT::vmax(g.q[0]) >= st.thr0) {
            if (st.n_deferred < kDefer) {
              slots.data[st.n_deferred * NT] = g.q[0];
              slots.index[st.n_deferred * NT] = v;
            }
            ++st.n_deferred;
          } else {
            acc_vector<BF16>(st.acc, g.q[0], st.c);
          }
          const uint4 t = g.q[0];
          g.q[0] = g.q[1]; g.q[1] = g.q[2]; g.q[2] = g.q[3]; g.q[3] = t;
          v += NT;
        }
      } else {
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
    // ---- segment boundary
    unsigned long long held;
    if (__any_sync(kFull, st.n_deferred > kDefer))
      held = resolve_by_rescan<BF16>(&sh, seg.row, seg.v0 + (int)threadIdx.x, seg.v1, pt.v_full, p.V, &st);
    else
      held = resolve_deferred<BF16>(&sh, slots, &st);
    publish_warp_sums(sh, st, held);
    const bool more = cur.valid;
    __syncthreads();
    const bool overflow = sh.cnt > kBufCap;
    const int split = blockIdx.x - (int)(((long long)seg.a * pt.vec_per_row) / pt.span);
    const size_t slot_id = (size_t)seg.a * p.max_splits + split;
    emit_partial(sh, p, slot_id, overflow);
    if (overflow)
      select_by_rescan<BF16>(K, p.V, pt.v_full, seg.row, seg.v0, seg.v1, p.part_keys + slot_id * K, sh.held);
    if (more)
      warmup_stage1<BF16>(sh, K, g, cur.tv0 + (int)threadIdx.x, cur.seg.v1, pt.v_full, ring + ((n + 1) & 1u) * 4 * NT);
    __syncthreads();
    if (!more) break;
    if (warp == 0) warmup_stage2(sh, K);
    __syncthreads();
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
  return 2 * 4 * (size_t)kExpandThreads * sizeof(uint4) + (size_t)kDefer * kExpandThreads * (sizeof(uint4) + sizeof(int)) +
         ((size_t)B + 1) * sizeof(int);
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
