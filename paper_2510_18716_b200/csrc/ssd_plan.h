// Work decomposition of one decode-attention launch, written once for host and device.
//
// The slots of a layer that hold a token form one logical stream, ordered by (sequence, head,
// slot).  The stream is cut into equal shares, one per worker (a warp); a worker walks its share
// in chunks of at most `chunk` slots that never cross a (sequence, head) boundary.  Inside one
// head's region the valid slots lie in up to three physically contiguous runs: the prompt, the
// static (top-M) set and the ring.  Everything here is 32-bit integer arithmetic on the layout
// tables; the kernel uses it to address its copies, and the host uses the same code to enumerate
// those copies for inspection (ssd_debug_decode_plan).
#pragma once

#include <stdint.h>

#if defined(__CUDACC__)
#define SSD_HD __host__ __device__ __forceinline__
#else
#define SSD_HD inline
#endif

namespace ssd {

constexpr int kPlanMaxHeads = 128;
constexpr int kShareAlign = 8;      // share boundaries are multiples of this many logical slots
constexpr int kMinShare = 16;       // shares are never cut smaller than this
constexpr int kPlanMaxWorkers = 32768;

// One head of a layer: x = first slot of the head inside a sequence's block, y = static capacity
// (M for semantic heads, 0 for spatial), z = ring capacity (R or W), w = 1 for semantic heads.
struct HeadRec {
  int32_t x, y, z, w;
};

// What a decode launch needs to know about the layer (passed by value to the kernel).
struct LayerView {
  int32_t H, L, n_seqs, seq_slots;  // seq_slots = physical slots per sequence in this layer
  int32_t prompt_valid;             // 0 or L
  int32_t static_valid;             // valid static slots of semantic heads
  int32_t t_img;                    // image tokens held; a spatial ring holds min(t_img, z) of them
  int32_t t_sem;                    // same count for semantic rings: t_img, or the tokens buffered since
                                    // the last re-selection when the ring is used as a row buffer
  int32_t contig;                   // 1 if every head's valid slots are one run from its first slot
  int32_t max_vh;                   // most valid slots any head holds
  int32_t cum[kPlanMaxHeads + 1];   // exclusive prefix of valid slots per head
  HeadRec head[kPlanMaxHeads];
};

// Ring slots of a head that hold a token.
SSD_HD int ring_valid(const LayerView& v, const HeadRec& d) {
  const int t = d.w ? v.t_sem : v.t_img;
  return t < d.z ? t : d.z;
}

SSD_HD int head_valid(const LayerView& v, int h) {
  const HeadRec d = v.head[h];
  return v.prompt_valid + (d.w ? v.static_valid : 0) + ring_valid(v, d);
}

// Fill the fields derived from the others: cum[], max_vh, contig.
inline void view_finish(LayerView& v);

// True if, for every head, the valid slots are physically contiguous from the head's first slot:
// the prompt is loaded (or there is none) and the static set of semantic heads is full.
inline bool view_contiguous(const LayerView& v) {
  if (v.prompt_valid != v.L) return false;
  for (int h = 0; h < v.H; ++h)
    if (v.head[h].w && v.static_valid != v.head[h].y) return false;
  return true;
}

inline void view_finish(LayerView& v) {
  int run = 0, mx = 0;
  for (int h = 0; h < v.H; ++h) {
    v.cum[h] = run;
    const int n = head_valid(v, h);
    run += n;
    if (n > mx) mx = n;
  }
  v.cum[v.H] = run;
  v.max_vh = mx;
  v.contig = view_contiguous(v) ? 1 : 0;
}

// How the stream of T valid slots is cut into W shares.  Share i starts at floor(i * T / W) rounded
// down to a multiple of kShareAlign; with T = q * W + r that is i * q + floor(i * r / W), which stays
// in 32 bits (i, r < W <= 2^15; T < 2^31) and needs one short division.
struct Split {
  int32_t T, W, q, r;
  float w_over_t;
};

inline Split make_split(long T, long W) {
  Split s;
  s.T = (int32_t)T;
  s.W = (int32_t)W;
  s.q = (int32_t)(T / W);
  s.r = (int32_t)(T % W);
  s.w_over_t = (float)W / (float)T;
  return s;
}

// Workers a launch over `total_valid` logical slots uses, given the most it may use.
inline long plan_workers(long total_valid, long max_workers) {
  long cap = total_valid / kMinShare;
  if (cap < 1) cap = 1;
  if (max_workers > kPlanMaxWorkers) max_workers = kPlanMaxWorkers;
  return max_workers < cap ? max_workers : cap;
}

SSD_HD int32_t share_start(const Split& s, int32_t i) {
  if (i >= s.W) return s.T;
  const uint32_t a = (uint32_t)i * (uint32_t)s.q + ((uint32_t)i * (uint32_t)s.r) / (uint32_t)s.W;
  return (int32_t)(a & ~(uint32_t)(kShareAlign - 1));
}

// Largest worker index whose share starts at or before logical slot g (0 <= g < T): a floating-
// point estimate, made exact by stepping while the neighbouring share starts disagree.
SSD_HD int32_t share_of(const Split& s, int32_t g) {
  int32_t i = (int32_t)((float)g * s.w_over_t);
  if (i > s.W - 1) i = s.W - 1;
  if (i < 0) i = 0;
  while (i > 0 && share_start(s, i) > g) --i;
  while (i + 1 < s.W && share_start(s, i + 1) <= g) ++i;
  return i;
}

// Position of a walk through a share: logical slot g, inside head `head` of sequence `seq`, at
// valid-slot index i of that head (which holds vh valid slots).
struct Walk {
  int32_t g, g_end;
  int32_t seq, head, i, vh;
};

SSD_HD void walk_init(Walk& w, const LayerView& v, int32_t g0, int32_t g1) {
  const int32_t vseq = v.cum[v.H];
  w.g = g0;
  w.g_end = g1;
  w.seq = g0 / vseq;
  const int r = g0 - w.seq * vseq;
  int lo = 0, hi = v.H;  // head with cum[head] <= r < cum[head + 1]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (v.cum[mid] <= r) lo = mid; else hi = mid;
  }
  w.head = lo;  // cum[lo] <= r < cum[lo + 1], so the head found is never an empty one
  w.i = r - v.cum[lo];
  w.vh = v.cum[lo + 1] - v.cum[lo];
}

// Slots of the chunk at the current position (0 only when the part being walked is exhausted).
SSD_HD int walk_chunk(const Walk& w, int chunk) {
  int n = w.g_end - w.g;
  if (n > w.vh - w.i) n = w.vh - w.i;
  if (n > chunk) n = chunk;
  return n;
}

SSD_HD void walk_advance(Walk& w, const LayerView& v, int n) {
  w.g += n;
  w.i += n;
  if (w.i >= w.vh && w.g < w.g_end) {
    w.i = 0;
    do {
      if (++w.head == v.H) { w.head = 0; ++w.seq; }
      w.vh = v.cum[w.head + 1] - v.cum[w.head];
    } while (w.vh == 0);
  }
}

// A worker's share [g_begin, g_end), walked in stream order.  If the head at the end of the share is
// cut by the share boundary (the next worker holds the rest of it), g_tail is where the worker's
// piece of that head starts (g_begin if the head began in an earlier share); g_tail == g_end when
// the last head is not cut.
struct Share {
  int32_t g_begin, g_end, g_tail;
};

SSD_HD Share share_plan(const LayerView& v, const Split& sp, int32_t wk) {
  Share s;
  s.g_begin = share_start(sp, wk);
  s.g_end = share_start(sp, wk + 1);
  s.g_tail = s.g_end;
  if (s.g_begin < s.g_end) {
    Walk w;
    walk_init(w, v, s.g_end - 1, s.g_end);
    const int32_t head_start = s.g_end - 1 - w.i;
    if (head_start + w.vh > s.g_end) s.g_tail = head_start > s.g_begin ? head_start : s.g_begin;
  }
  return s;
}

// Physical runs that make up valid slots [i, i + n) of head h.  emit(src, dst, len) is called once
// per run, in order: copy `len` slots from slot `src` (relative to the head's first slot) to slot
// `dst` of the chunk.  Runs that are physically adjacent are merged, so a head whose prompt and
// static set are full yields a single run.  The lengths add up to n.
#if defined(__CUDACC__)
#pragma nv_exec_check_disable
#endif
template <class Emit>
SSD_HD void chunk_runs(const LayerView& v, int h, int i, int n, Emit emit) {
  const HeadRec d = v.head[h];
  const int sv = d.w ? v.static_valid : 0;
  const int rv = ring_valid(v, d);
  const int l0[3] = {0, v.prompt_valid, v.prompt_valid + sv};  // logical start of each run
  const int ln[3] = {v.prompt_valid, sv, rv};
  const int p0[3] = {0, v.L, v.L + d.y};                       // physical start of each run
  int ps = 0, pd = 0, pl = 0;                                  // pending (not yet emitted) run
#if defined(__CUDA_ARCH__)
#pragma unroll
#endif
  for (int r = 0; r < 3; ++r) {
    const int a = i > l0[r] ? i : l0[r];
    const int b = i + n < l0[r] + ln[r] ? i + n : l0[r] + ln[r];
    if (b <= a) continue;
    const int s = p0[r] + (a - l0[r]);
    if (pl > 0 && ps + pl == s) {
      pl += b - a;
    } else {
      if (pl > 0) emit(ps, pd, pl);
      ps = s;
      pd = a - i;
      pl = b - a;
    }
  }
  if (pl > 0) emit(ps, pd, pl);
}

}  // namespace ssd
