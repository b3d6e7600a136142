// The expand pass: one streaming read of every active draft-logits row, giving per row the
// softmax normaliser and entropy sums and the K largest logits (ties to the lower token id)
//                                                        (Sec. 4.2.1, Eq. 2, Sec. 4.2.2).
//
// Work partition.  The active rows (a device-side count per sequence) are laid end to end as
// n_rows * vec_per_row 16-byte vectors and cut into contiguous spans of equal cost, one per WARP
// of a persistent grid (one CTA of 20 warps per SM).  A span may cover the tail of one row and
// the head of the next; each (row, warp) piece is a "segment" and produces one partial record.
// Opening a segment costs about as much as streaming kSegmentPad vectors, so the cut is even
// in vectors + kSegmentPad per row opened.
// The pruning kernel merges the partials of a row in double precision.  After one barrier at
// the start (the row list) the warps never wait for each other: while one warp is between
// segments the other 19 on the SM keep the memory pipe full.  (One CTA per SM rather than
// three smaller ones: the warps of an older CTA are served first, and its work would end early.)
//
// Data movement.  A warp works on groups of 128 consecutive vectors (2 KB), four per lane, 32
// apart, and owns kRingSlots shared-memory slots of 2 KB: while group n is in registers, groups
// n+1 .. n+kRingSlots are in flight, across segment boundaries too.  bf16 rows: each lane owns 4 x 16
// bytes of a slot, fills them with cp.async and reads back only what it copied itself, so the only
// wait is on its own copies (cp.async.wait_group).  fp32 rows: lane 0 fills a slot with ONE bulk copy
// (cp.async.bulk: the TMA unit moves the bytes and reports them to the slot's transaction barrier),
// the warp waits on the barrier (a bounded poll: a wait that runs out sets C2T_ST_INTERNAL instead of
// hanging), every lane takes its four vectors, and after a warp barrier the slot is requested again.
//
// Sums.  In base-2 units relative to a warp-uniform offset c = -m log2(e):  t = x log2(e) + c,
// S = sum 2^t, U = sum 2^t t  (one unpack, FMA, ex2, add, FMA per element).  m is the largest
// value the warp has met when c was last set, and only vectors whose elements are all below the
// filter (hence below m) are summed in the stream, so t <= 0.  (x log2(e) uses the fp32
// constant: a relative error of 1.3e-8 |x| in an element's weight, far inside tolerance.)
//
// Top-K.  A vector with an element at or above the filter is not summed but set aside in the
// warp's queue in shared memory (ballot-ranked places, so the order is fixed).  When the queue
// is nearly full, and at the end of the segment, the warp drains it, one element per lane and
// step: elements below the filter join the sums; the others join a small pool of keys next to
// the K largest keys found so far, the pool is ranked by counting, the K largest stay and the
// rest join the sums.  At the end of the segment all of the K largest but the first join the
// sums too: the segment's largest key stays out and is handed on exactly, so the sums keep fp32
// relative accuracy with respect to "everything but the maximum" however peaked the row is.
// The filter starts as the K-th largest lane maximum of the segment's first two groups (K
// distinct elements are at or above it) and after every drain is just above the K-th largest
// value so far: later elements of that value have higher token ids and lose the tie.
// Everything depends only on the warp's own data in a fixed order, so the results are
// reproducible bit for bit.
#include "vocab_common.cuh"
#include "level_prune.cuh"

namespace c2t {
namespace {

constexpr int kEWarps = kExpandThreads / 32;
constexpr int kVPL = kExpandVecPerLane;               // vectors of a group per lane, 32 apart
constexpr int kGroupVecs = 32 * kVPL;                 // vectors of one group of a warp
constexpr int kRingSlots = 2;                         // groups in flight per warp behind the one in registers (3 measured 3 % slower)
constexpr int kDrainAt = 12;                          // queued vectors that trigger a drain: early drains keep the filter tight
constexpr int kQueueCap = kDrainAt + kGroupVecs;      // a whole group always fits behind kDrainAt vectors

// What one warp owns in shared memory.
constexpr int kPool = 64;                             // keys ranked at a time (the K kept ones and up to 32 + 32 - K new)
struct WarpShared {
  uint4 ring[kRingSlots][kGroupVecs];
  unsigned long long mbar[kRingSlots];  // one transaction barrier per ring slot
  uint4 qdata[kQueueCap];
  int qindex[kQueueCap];
  unsigned long long pool[kPool];      // [0, K): the K largest keys so far, sorted (0 = none); behind them the new ones
  unsigned long long ranked[C2T_MAX_TOPK];
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

// the sums of one vector; t = x scale + c (scale is log2(e), or 0 to leave the vector out)
template <bool BF16>
__device__ __forceinline__ void acc_vector(Acc &a, const uint4 &q, float scale, float c) {
  float x[Vec<BF16>::N];
  Vec<BF16>::unpack(q, x);
#pragma unroll
  for (int i = 0; i < Vec<BF16>::N; i += 2) {
    const float t0 = fmaf(x[i], scale, c), t1 = fmaf(x[i + 1], scale, c);
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
  int qn;                     // warp-uniform: vectors in the queue
};

struct Group {
  uint4 q[kVPL];
};

// ---------------------------------------------------------------- segments of a span

// a / b for non-negative operands; the 32-bit division is much shorter when both fit
__device__ __forceinline__ long long div_floor(long long a, long long b) {
  if (((unsigned long long)(a | b) >> 32) == 0) return (long long)((unsigned)a / (unsigned)b);
  return a / b;
}

// Position x of the padded rows laid end to end -> position in the real rows laid end to end
// (a position inside a row's pad is the row's start).
__device__ __forceinline__ long long real_position(long long x, long long vrow, long long vtotal, int vpr) {
  if (x >= vtotal) x = vtotal;
  const long long row = div_floor(x, vrow);
  const long long off = x - row * vrow - kSegmentPad;
  return row * vpr + (off > 0 ? off : 0);
}


struct Segment {
  const char *row;
  int a, v0, v1;     // vectors [v0, v1) of active row a
};

struct SegWalk {
  int a, v0, left, vec_per_row;
  __device__ SegWalk(long long start, long long end, int vpr) : vec_per_row(vpr) {
    a = (int)div_floor(start, vpr);
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

__device__ __forceinline__ unsigned next_slot(unsigned slot) { return slot + 1 == kRingSlots ? 0u : slot + 1; }

// Two ways to fill a ring slot.  bf16 rows: every lane copies its own four vectors with cp.async and waits for its
// own copies (cp.async.wait_group); the kernel is bound by instruction issue there, and this form needs the fewest
// issue slots.  fp32 rows (half the elements per byte, so the memory side weighs more): one bulk copy per slot, below;
// measured on a 640-row level, bulk copies against cp.async: fp32 63.6 against 67.6 us, bf16 50 against 47.2 us.
template <int OFF>   // both addresses + OFF bytes
__device__ __forceinline__ void cp_async_16(uint32_t smem_dst, const void *gmem_src) {
  asm volatile("cp.async.cg.shared.global [%0 + %2], [%1 + %2], 16;" ::"r"(smem_dst), "l"(gmem_src), "n"(OFF) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// the lane's kVPL copies of a whole group / of a group cut off at vector lim
template <int U>
struct LaneCopies {
  static __device__ __forceinline__ void all(uint32_t dst, const uint4 *src) {
    LaneCopies<U - 1>::all(dst, src);
    cp_async_16<(U - 1) * 512>(dst, src);
  }
  static __device__ __forceinline__ void below(uint32_t dst, const uint4 *src, int vt, int lim) {
    LaneCopies<U - 1>::below(dst, src, vt, lim);
    if (vt + (U - 1) * 32 < lim) cp_async_16<(U - 1) * 512>(dst, src);
  }
};
template <>
struct LaneCopies<0> {
  static __device__ __forceinline__ void all(uint32_t, const uint4 *) {}
  static __device__ __forceinline__ void below(uint32_t, const uint4 *, int, int) {}
};

// A warp's ring of bulk copies: every slot is filled by ONE bulk copy (the TMA unit moves up to 2 KB from global to shared memory
// and reports the bytes to the slot's transaction barrier), issued by lane 0.  All lanes hold the same state.
constexpr int kRingWaitLimit = 1 << 22;               // polls of a barrier before the warp gives up (and says so)
struct Ring {
  uint32_t bar0;             // shared-memory address of the first slot's barrier; the others follow at 8 bytes
  uint32_t phase;            // bit s: parity of the phase slot s's next wait completes
  uint32_t pending;          // bit s: a copy into slot s was issued and has not been waited for
  __device__ __forceinline__ void init(WarpShared *ws, int lane) {
    bar0 = (uint32_t)__cvta_generic_to_shared(&ws->mbar[0]);
    phase = 0u;
    pending = 0u;
    if (lane == 0) {
#pragma unroll
      for (int i = 0; i < kRingSlots; ++i) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar0 + 8u * i) : "memory");
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
  }
  // n_vec whole vectors from src into the slot (lane 0 issues; the slot's last readers are behind a __syncwarp)
  __device__ __forceinline__ void issue(unsigned s, uint4 *slot, const uint4 *src, int n_vec, int lane) {
    if (n_vec <= 0) return;
    if (lane == 0) {
      const uint32_t bar = bar0 + 8u * s, bytes = (uint32_t)n_vec * 16u;
      const uint32_t dst = (uint32_t)__cvta_generic_to_shared(slot);
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
    }
    pending |= 1u << s;
  }
  // until the slot's copy (if one is outstanding) has landed; false if the wait ran out
  __device__ __forceinline__ bool wait(unsigned s) {
    if (!((pending >> s) & 1u)) return true;
    const uint32_t bar = bar0 + 8u * s, par = (phase >> s) & 1u;
    uint32_t done = 0u;
    for (int i = 0; i < kRingWaitLimit && !done; ++i)
      asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                   : "=r"(done) : "r"(bar), "r"(par) : "memory");
    phase ^= 1u << s;
    pending &= ~(1u << s);
    return done != 0u;
  }
};

// Requests the whole vectors of the cursor's group into a ring slot.
template <bool BULK>
__device__ __forceinline__ void prefetch_group(Ring &ring, unsigned s, const GroupCursor &c, uint4 *slot, int v_full, int lane) {
  if (c.valid) {
    const int lim = c.seg.v1 < v_full ? c.seg.v1 : v_full;
    if (BULK) {
      const int n = lim - c.tv0;
      ring.issue(s, slot, reinterpret_cast<const uint4 *>(c.seg.row) + c.tv0, n < kGroupVecs ? n : kGroupVecs, lane);
    } else {
      const uint4 *src = reinterpret_cast<const uint4 *>(c.seg.row) + c.tv0 + lane;
      const uint32_t dst = (uint32_t)__cvta_generic_to_shared(slot + lane);
      if (c.tv0 + kGroupVecs <= lim) LaneCopies<kVPL>::all(dst, src);
      else LaneCopies<kVPL>::below(dst, src, c.tv0 + lane, lim);
    }
  }
  if (!BULK) cp_async_commit();
}

// Until the copies into slot s have landed (cp.async: s is the oldest request, the only one ever waited for).
template <bool BULK>
__device__ __forceinline__ bool ring_wait(Ring &ring, unsigned s) {
  if (BULK) return ring.wait(s);
  cp_async_wait<kRingSlots - 1>();
  return true;
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
    for (int u = 0; u < kVPL; ++u) g.q[u] = slot[lane + u * 32];
  } else {
#pragma unroll
    for (int u = 0; u < kVPL; ++u) {
      const int v = vt + u * 32;
      g.q[u] = make_uint4(lo, lo, lo, lo);
      if (v < c.seg.v1) g.q[u] = v < v_full ? slot[lane + u * 32] : VT::load(c.seg.row, v, v_full, V);
    }
  }
#pragma unroll
  for (int u = 0; u < kVPL; ++u) VT::clamp(g.q[u]);
}

// ---------------------------------------------------------------- start of a segment

// the float just above the value of an orderable word
__device__ __forceinline__ float value_just_above(uint32_t orderable) {
  return __uint_as_float(f32_from_orderable(orderable + 1u));
}

// The filter and the reference of a new segment, from the lane maxima over its first two
// groups (the first is in registers, the second has landed in the ring: the caller has waited for it); TOPM: also the
// floor of the candidate collection (.z).
template <bool BF16, bool TOPM>
__device__ __noinline__ float4 segment_warmup(int K, Group g, int vt, int v1, int v_full, const uint4 *next_slot) {
  using VT = Vec<BF16>;
  const int lane = threadIdx.x & 31;
  float lmax = -INFINITY;
#pragma unroll
  for (int u = 0; u < kVPL; ++u) {
    if (vt + u * 32 < v1) {
      const float vm = VT::vmax(g.q[u]);
      if (vm == vm) lmax = fmaxf(lmax, vm);
    }
  }
  const int lim = v1 < v_full ? v1 : v_full;
#pragma unroll
  for (int u = 0; u < kVPL; ++u) {
    if (vt + kGroupVecs + u * 32 < lim) {  // same segment, whole vector: it is in the ring
      uint4 q = next_slot[lane + u * 32];
      VT::clamp(q);
      const float vm = VT::vmax(q);
      if (vm == vm) lmax = fmaxf(lmax, vm);
    }
  }
  uint32_t live = f32_orderable(__float_as_uint(lmax)), kth = 0, first = 0, low = 0;
  const int rounds = TOPM && K < kTopmRank ? kTopmRank : K;
  for (int r = 0; r < rounds; ++r) {       // K-th largest lane maximum
    const uint32_t cur = __reduce_max_sync(kFull, live);
    if (r == 0) first = cur;
    if (r == K - 1) kth = cur;
    if (TOPM && r == kTopmRank - 1) low = cur;
    const unsigned bal = __ballot_sync(kFull, live == cur);
    if (lane == __ffs(bal) - 1) live = 0;
  }
  const uint32_t none = f32_orderable(0xFF800000u);   // -inf: a lane without data
  float4 out;
  out.x = kth <= none ? -INFINITY : __uint_as_float(f32_from_orderable(kth));      // filter
  out.y = first <= none ? 0.f : __uint_as_float(f32_from_orderable(first));        // reference (any finite value if no data)
  out.z = low <= none ? kTopmLowestFloor : fmaxf(__uint_as_float(f32_from_orderable(low)), kTopmLowestFloor);
  out.w = 0.f;
  return out;
}

// ---------------------------------------------------------------- draining the queue

struct Drained {
  Acc acc;
  float c, m, thr;
};

// Empties the warp's queue, one element per lane and step.  Elements below the filter are
// summed.  The others are appended to the pool behind the K largest keys so far; whenever
// another step might not fit, and at the end, the pool is ranked by counting: the K largest
// keys stay (sorted, not summed yet), the rest is summed.
template <bool BF16>
__device__ __forceinline__ Drained drain_queue(WarpShared *ws, int qn, int K, Acc acc, float c, float m, float thr,
                                               uint32_t *status) {
  constexpr int EPV = Vec<BF16>::N;        // elements per vector
  constexpr int VPS = 32 / EPV;            // vectors per step
  const int lane = threadIdx.x & 31;
  const unsigned lt_mask = (1u << lane) - 1u;
  const int sub = lane / EPV, e = lane % EPV;
  int pn = K;
  for (int base = 0;; base += VPS) {
    const bool more = base < qn;
    if (!more || pn > kPool - 32) {
      // ---- rank the pool: lane l owns keys l and l + 32
      __syncwarp();
      const unsigned long long a = lane < pn ? ws->pool[lane] : 0ull;
      const unsigned long long b = lane + 32 < pn ? ws->pool[lane + 32] : 0ull;
      if (lane < K) ws->ranked[lane] = 0ull;
      int ra = 0, rb = 0;
      if (pn <= 32) {
#pragma unroll 4
        for (int r = 0; r < pn; ++r) ra += ws->pool[r] > a;
      } else {
#pragma unroll 4
        for (int r = 0; r < pn; ++r) {
          const unsigned long long kr = ws->pool[r];
          ra += kr > a;
          rb += kr > b;
        }
      }
      __syncwarp();
      // the reference follows the largest key before anything of the pool is summed
      const uint32_t top_hi = (a != 0ull && ra == 0) ? (uint32_t)(a >> 32) : ((b != 0ull && rb == 0) ? (uint32_t)(b >> 32) : 0u);
      const unsigned owner = __ballot_sync(kFull, top_hi != 0u);
      if (owner) {
        const float hm = __uint_as_float(f32_from_orderable(__shfl_sync(kFull, top_hi, __ffs(owner) - 1)));
        if (hm > m) {
          const float new_c = -hm * kLog2e;
          acc_rescale(acc, c, new_c);
          c = new_c;
          m = hm;
        }
      }
      if (a != 0ull) {
        if (ra < K) ws->ranked[ra] = a;
        else acc_scalar(acc, c, key_value(a));
      }
      if (b != 0ull) {
        if (rb < K) ws->ranked[rb] = b;
        else acc_scalar(acc, c, key_value(b));
      }
      __syncwarp();
      if (lane < K) ws->pool[lane] = ws->ranked[lane];
      pn = K;
      if (!more) break;
    }
    const int j = base + sub;
    bool cand = false;
    unsigned long long key = 0ull;
    if (j < qn) {
      float x;
      if (BF16) x = __uint_as_float((uint32_t)reinterpret_cast<const uint16_t *>(ws->qdata + j)[e] << 16);
      else x = reinterpret_cast<const float *>(ws->qdata + j)[e];
      cand = x >= thr;
      if (cand) key = make_key(x, (uint32_t)ws->qindex[j] * EPV + e);
      else acc_scalar(acc, c, x);                    // (a NaN element poisons the sums, as it must)
    }
    const unsigned mask = __ballot_sync(kFull, cand);
    if (cand && C2T_IN_BOUNDS(pn + __popc(mask & lt_mask), kPool, status)) ws->pool[pn + __popc(mask & lt_mask)] = key;
    pn += __popc(mask);
  }
  __syncwarp();
  // the list is exact for everything read so far: from now on only values above its K-th matter
  const unsigned long long kth = ws->pool[K - 1];
  if (kth != 0ull) thr = fmaxf(thr, value_just_above((uint32_t)(kth >> 32)));
  Drained d;
  d.acc = acc; d.c = c; d.m = m; d.thr = thr;
  return d;
}

// Candidates of the truncated entropy (Eq. 3): where a warp puts the vectors whose largest element reaches its
// segment's floor (ballot-ranked places in stream order, so the result does not depend on timing).
struct TopmState {
  uint4 *region;              // the warp's part of the pool
  int cap, n, first;          // its size in vectors; vectors set aside by the warp so far (may pass cap: then nothing more is stored); n when the segment began
  float floor;
  unsigned long long keep;    // L2 policy of the stores: the vectors are read back right after the pass, the rows never again
};

__device__ __forceinline__ void store_keep_in_l2(uint4 *dst, const uint4 &q, unsigned long long policy) {
  asm volatile("st.global.L2::cache_hint.v4.u32 [%0], {%1, %2, %3, %4}, %5;"
               ::"l"(dst), "r"(q.x), "r"(q.y), "r"(q.z), "r"(q.w), "l"(policy) : "memory");
}

// One group: vectors that meet the filter go to the queue, the others into the sums.  WHOLE:
// no lane is past the segment's end (a vector past it holds the lowest value, below every floor).
template <bool BF16, bool WHOLE, bool TOPM>
__device__ __forceinline__ void process_group(WarpShared *ws, const Group &g, SegState &st, TopmState &ts, int vt, int v1,
                                              unsigned lt_mask, uint32_t *status) {
  using VT = Vec<BF16>;
  float vm[kVPL];
#pragma unroll
  for (int u = 0; u < kVPL; ++u) vm[u] = VT::vmax(g.q[u]);
  if (TOPM) {
#pragma unroll
    for (int u = 0; u < kVPL; ++u) {
      const bool c = vm[u] >= ts.floor;              // (false for a vector with a NaN; such a row is reported anyway)
      const unsigned cm = __ballot_sync(kFull, c);
      const int pos = ts.n + __popc(cm & lt_mask);
      if (c && pos < ts.cap) store_keep_in_l2(ts.region + pos, g.q[u], ts.keep);
      ts.n += __popc(cm);
    }
  }
  float gm = vm[0];
#pragma unroll
  for (int u = 1; u < kVPL; ++u) gm = fmaxf(gm, vm[u]);
  const bool any_hit = gm >= st.thr;
  if (!__any_sync(kFull, any_hit)) {
#pragma unroll
    for (int u = 0; u < kVPL; ++u) acc_vector<BF16>(st.acc, g.q[u], kLog2e, st.c);
  } else {
    // The sums still run over all four vectors in one straight line; a vector that goes to the
    // queue is left out by t = 0 x - 200 (2^-200 flushes to zero and 0 * -200 adds nothing to U).
    bool hit[kVPL];
    unsigned mask[kVPL];
#pragma unroll
    for (int u = 0; u < kVPL; ++u) {
      hit[u] = vm[u] >= st.thr && (WHOLE || vt + u * 32 < v1);
      mask[u] = __ballot_sync(kFull, hit[u]);
    }
#pragma unroll
    for (int u = 0; u < kVPL; ++u) {
      if (hit[u]) {
        const int pos = st.qn + __popc(mask[u] & lt_mask);
        if (C2T_IN_BOUNDS(pos, kQueueCap, status)) {
          ws->qdata[pos] = g.q[u];
          ws->qindex[pos] = vt + u * 32;
        }
      }
      st.qn += __popc(mask[u]);
    }
#pragma unroll
    for (int u = 0; u < kVPL; ++u)
      acc_vector<BF16>(st.acc, g.q[u], hit[u] ? 0.f : kLog2e, hit[u] ? -200.f : st.c);
  }
}

template <bool BF16>
__device__ __forceinline__ void drain_into(WarpShared *ws, SegState &st, int K, uint32_t *status) {
  __syncwarp();                                      // the queue was written by other lanes
  const Drained d = drain_queue<BF16>(ws, st.qn, K, st.acc, st.c, st.m, st.thr, status);
  st.acc = d.acc; st.c = d.c; st.m = d.m; st.thr = d.thr;
  st.qn = 0;
  __syncwarp();
}

// ---------------------------------------------------------------- the kernel

// The pass itself: what every warp of the grid does (a warp returns when its span is done).
template <bool BF16, bool TOPM>
__device__ __forceinline__ void expand_pass_body(const PassParams &p, unsigned char *s_dyn) {
  using VT = Vec<BF16>;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  WarpShared *ws = reinterpret_cast<WarpShared *>(s_dyn) + warp;
  int *s_off = reinterpret_cast<int *>(s_dyn + kEWarps * sizeof(WarpShared));

  const int K = p.K;
  const int n_rows = build_row_offsets(p.counts, p.B, p.rows_per_seq_max, s_off);   // the only barriers
  if (blockIdx.x == 0 && p.row_off)                  // the pruning kernel finds a sequence's rows with this
    for (int i = threadIdx.x; i <= p.B; i += kExpandThreads) p.row_off[i] = s_off[i];
  const int vpr = (p.V + VT::N - 1) / VT::N, v_full = p.V / VT::N;
  // spans of equal cost: rows behind kSegmentPad virtual vectors each, laid end to end, cut evenly
  const long long vrow = (long long)vpr + kSegmentPad;
  const long long vtotal = (long long)n_rows * vrow;
  const long long workers = (long long)gridDim.x * kEWarps;
  long long span = div_floor(vtotal + workers - 1, workers);
  if (span < p.min_span) span = p.min_span;
  // consecutive workers sit on different SMs: a launch with few rows (level 0) still uses every SM
  const long long worker = (long long)warp * gridDim.x + blockIdx.x;
  if (worker == 0 && lane == 0) {
    p.info->n_rows = n_rows;
    p.info->vec_per_row = vpr;
    p.info->span = span;
    p.info->pad = kSegmentPad;
  }
  const long long start = real_position(worker * span, vrow, vtotal, vpr);
  const long long end = real_position((worker + 1) * span, vrow, vtotal, vpr);
  if (start >= end) return;

  const size_t esz = BF16 ? 2 : 4;
  GroupCursor cur(start, end, vpr, p, s_off, esz);   // the group being worked on
  GroupCursor pre = cur;                             // the group being requested, two ahead
  constexpr bool BULK = !BF16;                       // how the ring is filled (see above)
  Ring ring;
  ring.bar0 = ring.phase = ring.pending = 0u;
  if (BULK) ring.init(ws, lane);
  bool landed = true;                                // no wait for a copy has run out
#pragma unroll
  for (int i = 0; i < kRingSlots; ++i) {
    prefetch_group<BULK>(ring, i, pre, ws->ring[i], v_full, lane);
    pre.advance(p, s_off, esz);
  }
  unsigned n = 0;                                    // ring slot of the current group

  Group g;
  landed &= ring_wait<BULK>(ring, 0);
  take_group<BF16>(g, cur, ws->ring[0], v_full, p.V, lane);
  if (BULK) __syncwarp();                            // every lane has its vectors: the slot may be filled again
  prefetch_group<BULK>(ring, 0, pre, ws->ring[0], v_full, lane);
  pre.advance(p, s_off, esz);

  const unsigned lt_mask = (1u << lane) - 1u;
  SegState st;
  TopmState ts;
  ts.region = nullptr; ts.cap = 0; ts.n = 0; ts.first = 0; ts.floor = INFINITY; ts.keep = 0ull;
  if (TOPM) {
    asm("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(ts.keep));
    const long long busy = div_floor(vtotal + span - 1, span);       // workers with a span of this launch
    const long long cap = div_floor(p.topm_pool_vecs, busy > 0 ? busy : 1);
    ts.cap = (int)(cap < 0x3FFFFFFF ? cap : 0x3FFFFFFF);
    ts.region = p.topm_pool + worker * ts.cap;
  }
  bool fresh = true;                                 // the current group opens a segment
  for (;;) {
    const Segment seg = cur.seg;
    if (fresh) {
      landed &= ring_wait<BULK>(ring, next_slot(n));   // the group after this one
      const float4 w = segment_warmup<BF16, TOPM>(K, g, cur.tv0 + lane, seg.v1, v_full, ws->ring[next_slot(n)]);
      if (TOPM) { ts.floor = w.z; ts.first = ts.n; }
      st.acc.S0 = st.acc.S1 = st.acc.U0 = st.acc.U1 = 0.f;
      st.thr = w.x;
      st.m = w.y;
      st.c = -w.y * kLog2e;
      st.qn = 0;
      if (lane < K) ws->pool[lane] = 0ull;
      fresh = false;
    }
    // ---- the inside of a segment: this group, the next one (in the ring) and the one to be
    // requested (kRingSlots + 1 ahead) are whole groups of this segment, so nothing needs checking
    if (pre.valid && pre.seg.a == seg.a) {
      const int lim = seg.v1 < v_full ? seg.v1 : v_full;
      const int k = (lim - cur.tv0) / kGroupVecs - (kRingSlots + 1);
      if (k > 0) {
        const uint4 *src = reinterpret_cast<const uint4 *>(seg.row) + pre.tv0 + (BULK ? 0 : lane);
        int vt = cur.tv0 + lane;
        for (int i = 0; i < k; ++i) {
          process_group<BF16, true, TOPM>(ws, g, st, ts, vt, 0, lt_mask, p.status);
          n = next_slot(n);
          vt += kGroupVecs;
          landed &= ring_wait<BULK>(ring, n);
          uint4 *slot = ws->ring[n];
#pragma unroll
          for (int u = 0; u < kVPL; ++u) g.q[u] = slot[lane + u * 32];
#pragma unroll
          for (int u = 0; u < kVPL; ++u) VT::clamp(g.q[u]);
          if (BULK) {
            __syncwarp();
            ring.issue(n, slot, src, kGroupVecs, lane);
          } else {
            LaneCopies<kVPL>::all((uint32_t)__cvta_generic_to_shared(slot + lane), src);
            cp_async_commit();
          }
          src += kGroupVecs;
          if (st.qn > kDrainAt) drain_into<BF16>(ws, st, K, p.status);
        }
        cur.tv0 += k * kGroupVecs;
        pre.tv0 += (k - 1) * kGroupVecs;             // the last step may leave the segment
        pre.advance(p, s_off, esz);
      }
    }
    // ---- one group near the end of a segment, everything checked
    const int vt = cur.tv0 + lane;
    process_group<BF16, false, TOPM>(ws, g, st, ts, vt, seg.v1, lt_mask, p.status);
    const bool last = cur.last_of_segment();
    cur.advance(p, s_off, esz);
    n = next_slot(n);
    if (cur.valid) {                                 // next group (of this or of the next segment) into registers
      landed &= ring_wait<BULK>(ring, n);
      uint4 *slot = ws->ring[n];
      take_group<BF16>(g, cur, slot, v_full, p.V, lane);
      if (BULK) __syncwarp();
      prefetch_group<BULK>(ring, n, pre, slot, v_full, lane);
      pre.advance(p, s_off, esz);
    }
    if (last || st.qn > kDrainAt) drain_into<BF16>(ws, st, K, p.status);
    if (last) {
      // ---- the segment's record: the K largest keys but the first join the sums; sums in a
      // fixed order, the sorted keys, the held-out head
      const unsigned long long mine = lane < K ? ws->pool[lane] : 0ull;
      if (lane > 0 && mine != 0ull) acc_scalar(st.acc, st.c, key_value(mine));
      float S = st.acc.S0 + st.acc.S1, U = st.acc.U0 + st.acc.U1;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        S += __shfl_down_sync(kFull, S, o);
        U += __shfl_down_sync(kFull, U, o);
      }
      const long long split = worker - div_floor((long long)seg.a * vrow + kSegmentPad, span);   // workers before the row's first
      const size_t slot_id = (size_t)seg.a * p.max_splits + (size_t)split;
      const unsigned have = __ballot_sync(kFull, mine != 0ull);
      const bool slot_ok = C2T_IN_BOUNDS(slot_id, p.n_slots, p.status);
      if (lane < K && slot_ok) p.part_keys[slot_id * K + lane] = mine;
      if (lane == 0 && slot_ok) {
        p.part_held[slot_id] = mine;
        p.part_stats[slot_id] = make_float4(st.c, S, U, __int_as_float(__popc(have)));
        if (TOPM) {
          TopmSegment rec;
          rec.first = (int)(worker * ts.cap) + ts.first;
          rec.n = ts.n > ts.cap ? -1 : ts.n - ts.first;
          rec.floor = ts.floor;
          rec.pad = 0;
          p.topm_seg[slot_id] = rec;
        }
      }
      __syncwarp();
      if (!cur.valid) break;
      fresh = true;
    }
  }
  // (every bulk copy that was issued has been waited for: the requests never run past the span)
  if (!BULK) cp_async_wait<0>();
  if (!landed && lane == 0 && p.status) atomicOr(p.status, C2T_ST_INTERNAL);
}

template <bool BF16, bool TOPM>
__global__ void __launch_bounds__(kExpandThreads, kExpandCtasPerSm) expand_pass_kernel(PassParams p) {
  extern __shared__ __align__(16) unsigned char s_dyn[];
  chain_enter();
  expand_pass_body<BF16, TOPM>(p, s_dyn);
}

// Expand and prune of a level in one launch, for small batches: the CTA that finishes last (an atomic ticket, nobody
// waits) has every row's partial records in front of it and does the per-sequence work of c2t_prune for all
// sequences, one after the other.
template <bool BF16>
__global__ void __launch_bounds__(kExpandThreads, kExpandCtasPerSm) expand_prune_kernel(PassParams p, TreeState t, int level,
                                                                                        c2t_frontier out) {
  extern __shared__ __align__(16) unsigned char s_dyn[];
  __shared__ unsigned s_ticket;
  chain_enter();
  expand_pass_body<BF16, false>(p, s_dyn);
  __threadfence();                                   // this CTA's records, before its ticket
  __syncthreads();
  if (threadIdx.x == 0) s_ticket = atomicAdd(t.ticket, 1u);
  __syncthreads();
  if (s_ticket != gridDim.x - 1) return;
  __threadfence();                                   // the other CTAs' records, after their tickets
  if (threadIdx.x == 0) *t.ticket = 0u;              // for the next launch
  // the pass's shared memory is free now
  static_assert(sizeof(PruneShared<kEWarps>) <= kEWarps * sizeof(WarpShared), "the prune's scratch must fit the warps' areas");
  PruneShared<kEWarps> &sh = *reinterpret_cast<PruneShared<kEWarps> *>(s_dyn);
  for (int b = 0; b < t.B; ++b) prune_level_body<kExpandThreads, false>(t, level, out, nullptr, 0, b, sh);
}

}  // namespace

int expand_min_span(int vocab, int elem_bytes, int K) {
  const int vec = 16 / elem_bytes;
  const int vec_per_row = (vocab + vec - 1) / vec;
  int lists = kStageKeys / (K < 1 ? 1 : K) - 1;      // one list in reserve: a row's pieces may start mid-worker
  lists = lists > 31 ? 31 : (lists < 4 ? 4 : lists);
  const int span = (vec_per_row + kSegmentPad + lists - 1) / lists;
  return span < 256 ? 256 : span;
}

size_t topm_pool_vectors(size_t batch, size_t rows_per_seq, int vocab, int elem_bytes) {
  const size_t vec = 16 / elem_bytes;
  const size_t n = batch * rows_per_seq * ((vocab + vec - 1) / vec) / kTopmPoolDivisor + 4096;
  return n < 0x7FFFFFFFu ? n : 0x7FFFFFFFu;          // records hold 32-bit positions
}

int max_splits_for(int vocab, int elem_bytes, int workers, int pad, int min_span) {
  const int vec = 16 / elem_bytes;
  const int vec_per_row = (vocab + vec - 1) / vec;
  int by_span = (vec_per_row + pad + min_span - 1) / min_span;
  if (by_span > workers) by_span = workers;
  return by_span + 1;
}

static size_t expand_dynamic_smem(int B) {
  return (size_t)kEWarps * sizeof(WarpShared) + ((size_t)B + 1) * sizeof(int);
}

cudaError_t prepare_expand_pass() {
  const int bytes = (int)expand_dynamic_smem(C2T_MAX_BATCH);
  const int fused = (int)expand_dynamic_smem(C2T_FUSED_MAX_BATCH);
  cudaError_t e = cudaFuncSetAttribute(expand_pass_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(expand_pass_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(expand_pass_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(expand_pass_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(expand_prune_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, fused);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(expand_prune_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, fused);
  return e;
}

cudaError_t launch_expand_prune(const PassParams &p, const TreeState &t, int level, const c2t_frontier *out, int dtype,
                                int grid, cudaStream_t s) {
  c2t_frontier o = {nullptr, nullptr, nullptr, nullptr};
  if (out) o = *out;
  const size_t smem = expand_dynamic_smem(p.B);
  if (dtype == C2T_BF16)
    return launch_chained(expand_prune_kernel<true>, dim3(grid), dim3(kExpandThreads), smem, s, p, t, level, o);
  return launch_chained(expand_prune_kernel<false>, dim3(grid), dim3(kExpandThreads), smem, s, p, t, level, o);
}

cudaError_t launch_expand_pass(const PassParams &p, int dtype, int grid, cudaStream_t s) {
  const size_t smem = expand_dynamic_smem(p.B);
  const bool bf16 = dtype == C2T_BF16;
  if (p.topm_pool) {                                 // also sets the candidates of Eq. 3 aside
    if (bf16) return launch_chained(expand_pass_kernel<true, true>, dim3(grid), dim3(kExpandThreads), smem, s, p);
    return launch_chained(expand_pass_kernel<false, true>, dim3(grid), dim3(kExpandThreads), smem, s, p);
  }
  if (bf16) return launch_chained(expand_pass_kernel<true, false>, dim3(grid), dim3(kExpandThreads), smem, s, p);
  return launch_chained(expand_pass_kernel<false, false>, dim3(grid), dim3(kExpandThreads), smem, s, p);
}

}  // namespace c2t
