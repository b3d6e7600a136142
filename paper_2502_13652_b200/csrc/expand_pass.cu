// The expand pass: one streaming read of every active draft-logits row, giving per row the
// softmax normaliser and entropy sums and the K largest logits (ties to the lower token id)
//                                                        (Sec. 4.2.1, Eq. 2, Sec. 4.2.2).
//
// Work partition.  The active rows (a device-side count per sequence) are laid end to end as
// n_rows * vec_per_row 16-byte vectors and cut into equal contiguous spans, one per WARP of a
// persistent grid (three CTAs of eight warps per SM).  A span may cover the tail of one row and
// the head of the next; each (row, warp) piece is a "segment" and produces one partial record.
// The pruning kernel merges the partials of a row in double precision.  After one barrier at
// the start (the row list) the warps never wait for each other: while one warp is between
// segments the other 23 on the SM keep the memory pipe full.
//
// Data movement.  A warp works on groups of 128 consecutive vectors (2 KB), four per lane, 32
// apart.  Each lane owns 4 x 16 bytes in each of two shared-memory slots and fills them with
// cp.async: while group n is in registers, groups n+1 and n+2 are in flight, across segment
// boundaries too.  A lane reads back only what it copied itself, so the only wait is on its own
// copies (cp.async.wait_group).
//
// Sums.  In base-2 units relative to a warp-uniform offset c = -m log2(e):  t = x log2(e) + c,
// S = sum 2^t, U = sum 2^t t  (one unpack, FMA, ex2, add, FMA per element).  m is the largest
// value the warp has met when c was last set, and only vectors whose elements are all below the
// filter (hence below m) are summed in the stream, so t <= 0.  (x log2(e) uses the fp32
// constant: a relative error of 1.3e-8 |x| in an element's weight, far inside tolerance.)
//
// Top-K.  A vector with an element at or above the filter is not summed but set aside in the
// warp's queue in shared memory (ballot-ranked places, so the order is fixed).  When the queue
// is nearly full, and at the end of the segment, the warp drains it: the elements go, one per
// lane, into the warp's sorted list of the 32 largest keys so far (one key per lane, insertion
// by shuffle) and into the sums; the largest key of the segment stays out of the sums and is
// handed on exactly, so the sums keep fp32 relative accuracy with respect to "everything but
// the maximum" however peaked the row is.  The filter starts as the K-th largest lane maximum
// of the segment's first two groups (K distinct elements are at or above it) and after every
// drain is just above the K-th largest value so far: later elements of that value have higher
// token ids and lose the tie.  Everything depends only on the warp's own data in a fixed
// order, so the results are reproducible bit for bit.
#include "vocab_common.cuh"

namespace c2t {
namespace {

constexpr int kEWarps = kExpandThreads / 32;
constexpr int kGroupVecs = 128;                       // vectors of one group of a warp
constexpr int kQueueCap = 160;                        // vectors a warp can set aside before it must drain
constexpr int kDrainAt = kQueueCap - kGroupVecs;      // a group always fits behind this many

// What one warp owns in shared memory.
struct WarpShared {
  uint4 ring[2][kGroupVecs];
  uint4 qdata[kQueueCap];
  int qindex[kQueueCap];
};

// ---------------------------------------------------------------- sums

struct Acc {
  float S0, S1, U0, U1;
};

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

// ---------------------------------------------------------------- per-warp state of a segment

struct SegState {
  Acc acc;                    // per lane
  float c;                    // warp-uniform offset of the sums, -m log2(e)
  float m;                    // warp-uniform reference value
  float thr;                  // warp-uniform filter
  unsigned long long mine;    // lane r: the r-th largest key drained so far (0 = none)
  int qn;                     // warp-uniform: vectors in the queue
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
  __device__ SegWalk(long long start, long long end, int vpr) : vec_per_row(vpr) {
    a = (int)(start / vpr);
    v0 = (int)(start - (long long)a * vpr);
    left = (int)(end - start);
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

// The groups of a warp's span in order; all lanes hold the same cursor.
struct GroupCursor {
  SegWalk walk;
  Segment seg;     // the segment the current group belongs to
  int tv0;         // first vector of the current group; the lane's are tv0 + lane + 32 u
  bool valid;
  __device__ GroupCursor(long long start, long long end, int vpr, const PassParams &p, const int *s_off, size_t esz)
      : walk(start, end, vpr) {
    seg = walk.take(p, s_off, esz);
    tv0 = seg.v0;
    valid = true;
  }
  __device__ bool last_of_segment() const { return tv0 + kGroupVecs >= seg.v1; }
  __device__ void advance(const PassParams &p, const int *s_off, size_t esz) {
    tv0 += kGroupVecs;
    if (tv0 >= seg.v1) {
      if (walk.done()) { valid = false; return; }
      seg = walk.take(p, s_off, esz);
      tv0 = seg.v0;
    }
  }
};

// ---------------------------------------------------------------- asynchronous prefetch ring

__device__ __forceinline__ void cp_async_16(void *smem_dst, const void *gmem_src) {
  const uint32_t dst = (uint32_t)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Requests the whole vectors of the cursor's group into the lane's places of a ring slot.
__device__ __forceinline__ void prefetch_group(const GroupCursor &c, uint4 *slot, int v_full, int lane) {
  if (c.valid) {
    const int lim = c.seg.v1 < v_full ? c.seg.v1 : v_full;
    const uint4 *src = reinterpret_cast<const uint4 *>(c.seg.row) + c.tv0 + lane;
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (c.tv0 + lane + u * 32 < lim) cp_async_16(slot + lane + u * 32, src + u * 32);
  }
  cp_async_commit();
}

// Takes the cursor's group out of a ring slot (its copies have completed) into registers and
// clamps it.  Vectors past the segment end become -2^127, which adds exactly 0 to the sums; a
// ragged last vector of a row is assembled from scalar loads.
template <bool BF16>
__device__ __forceinline__ void take_group(Group &g, const GroupCursor &c, const uint4 *slot, int v_full, int V,
                                           int lane) {
  using VT = Vec<BF16>;
  const uint32_t lo = BF16 ? kLowestBf16x2 : __float_as_uint(kLowestF32);
  const int vt = c.tv0 + lane;
  if (c.tv0 + kGroupVecs <= (c.seg.v1 < v_full ? c.seg.v1 : v_full)) {
#pragma unroll
    for (int u = 0; u < 4; ++u) g.q[u] = slot[lane + u * 32];
  } else {
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int v = vt + u * 32;
      g.q[u] = make_uint4(lo, lo, lo, lo);
      if (v < c.seg.v1) g.q[u] = v < v_full ? slot[lane + u * 32] : VT::load(c.seg.row, v, v_full, V);
    }
  }
#pragma unroll
  for (int u = 0; u < 4; ++u) VT::clamp(g.q[u]);
}

// ---------------------------------------------------------------- start of a segment

// the float just above the value of an orderable word
__device__ __forceinline__ float value_just_above(uint32_t orderable) {
  return __uint_as_float(f32_from_orderable(orderable + 1u));
}

// The filter and the reference of a new segment, from the lane maxima over its first two
// groups (the first is in registers, the second has just landed in the ring).
template <bool BF16>
__device__ __noinline__ float2 segment_warmup(int K, Group g, int vt, int v1, int v_full, const uint4 *next_slot) {
  using VT = Vec<BF16>;
  const int lane = threadIdx.x & 31;
  float lmax = -INFINITY;
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    if (vt + u * 32 < v1) {
      const float vm = VT::vmax(g.q[u]);
      if (vm == vm) lmax = fmaxf(lmax, vm);
    }
  }
  cp_async_wait<1>();                      // the group after this one (all but the newest request)
  const int lim = v1 < v_full ? v1 : v_full;
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    if (vt + kGroupVecs + u * 32 < lim) {  // same segment, whole vector: it is in the ring
      uint4 q = next_slot[lane + u * 32];
      VT::clamp(q);
      const float vm = VT::vmax(q);
      if (vm == vm) lmax = fmaxf(lmax, vm);
    }
  }
  uint32_t live = f32_orderable(__float_as_uint(lmax)), kth = 0, first = 0;
  for (int r = 0; r < K; ++r) {            // K-th largest lane maximum
    kth = __reduce_max_sync(kFull, live);
    if (r == 0) first = kth;
    const unsigned bal = __ballot_sync(kFull, live == kth);
    if (lane == __ffs(bal) - 1) live = 0;
  }
  const uint32_t none = f32_orderable(0xFF800000u);   // -inf: a lane without data
  float2 out;
  out.x = kth <= none ? -INFINITY : __uint_as_float(f32_from_orderable(kth));      // filter
  out.y = first <= none ? 0.f : __uint_as_float(f32_from_orderable(first));        // reference (any finite value if no data)
  return out;
}

// ---------------------------------------------------------------- draining the queue

__device__ __forceinline__ unsigned long long shfl_key(unsigned long long k, int src) {
  return __shfl_sync(kFull, k, src);
}

__device__ __forceinline__ unsigned long long warp_max_key(unsigned long long k) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const unsigned long long other = __shfl_xor_sync(kFull, k, o);
    k = other > k ? other : k;
  }
  return k;
}

struct Drained {
  Acc acc;
  float c, m, thr;
  unsigned long long mine;
};

// Empties the warp's queue, one element per lane and step: every element is summed except the
// largest key of the segment so far (the head of the list), and the elements that beat the
// K-th key of the list are inserted into it.
template <bool BF16>
__device__ __noinline__ Drained drain_queue(const WarpShared *ws, int qn, int K, Acc acc, float c, float m, float thr,
                                            unsigned long long mine) {
  constexpr int EPV = Vec<BF16>::N;        // elements per vector
  constexpr int VPS = 32 / EPV;            // vectors per step
  const int lane = threadIdx.x & 31;
  const int sub = lane / EPV, e = lane % EPV;

  // the largest key in the queue
  unsigned long long best = 0ull;
  for (int base = 0; base < qn; base += VPS) {
    const int j = base + sub;
    if (j < qn) {
      float x;
      if (BF16) x = __uint_as_float((uint32_t)reinterpret_cast<const uint16_t *>(ws->qdata + j)[e] << 16);
      else x = reinterpret_cast<const float *>(ws->qdata + j)[e];
      const unsigned long long key = make_key(x, (uint32_t)ws->qindex[j] * EPV + e);
      if (x == x && key > best) best = key;
    }
  }
  const unsigned long long qmax = warp_max_key(best);
  const unsigned long long old_head = shfl_key(mine, 0);
  const unsigned long long head = qmax > old_head ? qmax : old_head;
  if (head != 0ull) {
    const float hm = key_value(head);
    if (hm > m) {                          // the reference rises: bring the sums along
      const float new_c = -hm * kLog2e;
      acc_rescale(acc, c, new_c);
      c = new_c;
      m = hm;
    }
  }
  // the previous head is no longer the maximum: it joins the sums
  if (old_head != 0ull && head != old_head && lane == 0) acc_scalar(acc, c, key_value(old_head));

  unsigned long long kth = shfl_key(mine, K - 1);
  for (int base = 0; base < qn; base += VPS) {
    const int j = base + sub;
    unsigned long long key = 0ull;
    if (j < qn) {
      float x;
      if (BF16) x = __uint_as_float((uint32_t)reinterpret_cast<const uint16_t *>(ws->qdata + j)[e] << 16);
      else x = reinterpret_cast<const float *>(ws->qdata + j)[e];
      const unsigned long long k = make_key(x, (uint32_t)ws->qindex[j] * EPV + e);
      if (k != head) acc_scalar(acc, c, x);          // (a NaN element poisons the sums, as it must)
      if (x == x) key = k;
    }
    unsigned cand = __ballot_sync(kFull, key > kth);
    while (cand) {
      const int src = __ffs(cand) - 1;
      cand &= cand - 1;
      const unsigned long long k = shfl_key(key, src);
      unsigned long long up = __shfl_up_sync(kFull, mine, 1);
      if (lane == 0) up = ~0ull;
      if (k > mine) mine = k > up ? up : k;          // place k, or take over the neighbour's key
    }
    kth = shfl_key(mine, K - 1);
  }
  // all of the K largest so far are in the list: from now on only values above its K-th matter
  if (kth != 0ull) thr = fmaxf(thr, value_just_above((uint32_t)(kth >> 32)));
  Drained d;
  d.acc = acc; d.c = c; d.m = m; d.thr = thr; d.mine = mine;
  return d;
}

// ---------------------------------------------------------------- the kernel

template <bool BF16>
__global__ void __launch_bounds__(kExpandThreads, kExpandCtasPerSm) expand_pass_kernel(PassParams p) {
  using VT = Vec<BF16>;
  extern __shared__ __align__(16) unsigned char s_dyn[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  WarpShared *ws = reinterpret_cast<WarpShared *>(s_dyn) + warp;
  int *s_off = reinterpret_cast<int *>(s_dyn + kEWarps * sizeof(WarpShared));

  const int K = p.K;
  const int n_rows = build_row_offsets(p.counts, p.B, p.rows_per_seq_max, s_off);   // the only barriers
  const int vpr = (p.V + VT::N - 1) / VT::N, v_full = p.V / VT::N;
  const long long total = (long long)n_rows * vpr;
  const long long workers = (long long)gridDim.x * kEWarps;
  long long span = (total + workers - 1) / workers;
  if (span < kMinSpanVectors) span = kMinSpanVectors;
  const long long worker = (long long)blockIdx.x * kEWarps + warp;
  if (worker == 0 && lane == 0) {
    p.info->n_rows = n_rows;
    p.info->vec_per_row = vpr;
    p.info->span = span;
  }
  const long long start = worker * span;
  const long long end = start + span < total ? start + span : total;
  if (start >= end) return;

  const size_t esz = BF16 ? 2 : 4;
  GroupCursor cur(start, end, vpr, p, s_off, esz);   // the group being worked on
  GroupCursor pre = cur;                             // the group being requested, two ahead
  prefetch_group(pre, ws->ring[0], v_full, lane);
  pre.advance(p, s_off, esz);
  prefetch_group(pre, ws->ring[1], v_full, lane);
  pre.advance(p, s_off, esz);
  unsigned n = 0;                                    // index of the current group: its ring slot is n & 1

  Group g;
  cp_async_wait<1>();
  take_group<BF16>(g, cur, ws->ring[0], v_full, p.V, lane);
  prefetch_group(pre, ws->ring[0], v_full, lane);
  pre.advance(p, s_off, esz);

  const unsigned lt_mask = (1u << lane) - 1u;
  SegState st;
  bool fresh = true;                                 // the current group opens a segment
  for (;;) {
    const Segment seg = cur.seg;
    const int vt = cur.tv0 + lane;
    if (fresh) {
      const float2 w = segment_warmup<BF16>(K, g, vt, seg.v1, v_full, ws->ring[(n + 1) & 1u]);
      st.acc.S0 = st.acc.S1 = st.acc.U0 = st.acc.U1 = 0.f;
      st.thr = w.x;
      st.m = w.y;
      st.c = -w.y * kLog2e;
      st.mine = 0ull;
      st.qn = 0;
      fresh = false;
    }
    // ---- one group: vectors that meet the filter go to the queue, the others into the sums
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const bool hit = VT::vmax(g.q[u]) >= st.thr && vt + u * 32 < seg.v1;
      const unsigned mask = __ballot_sync(kFull, hit);
      if (mask) {
        if (hit) {
          const int pos = st.qn + __popc(mask & lt_mask);
          ws->qdata[pos] = g.q[u];
          ws->qindex[pos] = vt + u * 32;
          const uint32_t lo = BF16 ? kLowestBf16x2 : __float_as_uint(kLowestF32);
          g.q[u] = make_uint4(lo, lo, lo, lo);       // adds exactly 0 below
        }
        st.qn += __popc(mask);
      }
      acc_vector<BF16>(st.acc, g.q[u], st.c);
    }
    const bool last = cur.last_of_segment();
    cur.advance(p, s_off, esz);
    ++n;
    if (cur.valid) {                                 // next group (of this or of the next segment) into registers
      cp_async_wait<1>();
      uint4 *slot = ws->ring[n & 1u];
      take_group<BF16>(g, cur, slot, v_full, p.V, lane);
      prefetch_group(pre, slot, v_full, lane);
      pre.advance(p, s_off, esz);
    }
    if (last || st.qn > kDrainAt) {
      __syncwarp();                                  // the queue was written by other lanes
      const Drained d = drain_queue<BF16>(ws, st.qn, K, st.acc, st.c, st.m, st.thr, st.mine);
      st.acc = d.acc; st.c = d.c; st.m = d.m; st.thr = d.thr; st.mine = d.mine;
      st.qn = 0;
      __syncwarp();
    }
    if (last) {
      // ---- the segment's record: sums in a fixed order, the sorted keys, the held-out head
      float S = st.acc.S0 + st.acc.S1, U = st.acc.U0 + st.acc.U1;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        S += __shfl_down_sync(kFull, S, o);
        U += __shfl_down_sync(kFull, U, o);
      }
      const long long split = worker - ((long long)seg.a * vpr) / span;
      const size_t slot_id = (size_t)seg.a * p.max_splits + (size_t)split;
      const unsigned have = __ballot_sync(kFull, st.mine != 0ull && lane < K);
      if (lane < K) p.part_keys[slot_id * K + lane] = st.mine;
      if (lane == 0) {
        p.part_held[slot_id] = st.mine;
        p.part_stats[slot_id] = make_float4(st.c, S, U, __int_as_float(__popc(have)));
      }
      if (!cur.valid) break;
      fresh = true;
    }
  }
  cp_async_wait<0>();
}

}  // namespace

int max_splits_for(int vocab, int elem_bytes, int workers) {
  const int vec = 16 / elem_bytes;
  const int vec_per_row = (vocab + vec - 1) / vec;
  int by_span = (vec_per_row + kMinSpanVectors - 1) / kMinSpanVectors;
  if (by_span > workers) by_span = workers;
  return by_span + 1;
}

static size_t expand_dynamic_smem(int B) {
  return (size_t)kEWarps * sizeof(WarpShared) + ((size_t)B + 1) * sizeof(int);
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
