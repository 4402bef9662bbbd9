// Single-token decode attention over the head-decoupled compressed KV store, and the
// per-step append/evict.
//
// Decode (consumer of Algorithm 1's output): for every (sequence, head) of one layer,
//   out = sum_i softmax_i(scale * <q, K_i>) V_i   over the slots that hold a token.
// It is a GEMV per head (1 flop per byte), so the kernel is built around keeping HBM busy and
// the instruction count per byte low, not around tensor cores:
//   * one CTA per SM, every streaming warp an independent worker.  The valid slots of the whole
//     layer form one logical stream of 512-byte slots ([K row | V row]) that is cut into equal
//     shares, one per worker, regardless of head type or length, so every SM moves the same bytes;
//   * a worker owns a ring of shared-memory stages.  Lane 0 fills them with bulk asynchronous
//     copies (cp.async.bulk, completion counted on an mbarrier per stage), one chunk of up to
//     kChunk slots per stage, and runs kStages chunks ahead of the arithmetic across head
//     boundaries; the query row of a head travels with the head's first chunk.  A stage is
//     pulled into registers and handed back to the copy engine before the arithmetic starts;
//   * arithmetic per chunk: the warp works as four groups of 8 lanes, group g taking slots g,
//     g + 4, ...; a lane covers 16 of the 128 dimensions with two 128-bit reads per row, packed
//     two-wide fp32 FMAs, three shuffles per dot product, and an online softmax in fp32 (base-2
//     exponent, scale folded into q);
//   * a head that lies inside one share is finished in registers.  A head cut by a share boundary
//     leaves a partial (m, l, acc[128]) in the worker's shared-memory mailbox.  Workers of a CTA
//     hold consecutive shares, so the pieces of such a head usually all belong to one CTA: the
//     worker that posts the last of them (shared-memory arrival counter, nobody waits) merges
//     them in worker order and writes the output.  For the at most two heads that cross the CTA's
//     own range, that worker hands the CTA's merged partial to an extra finisher warp, which
//     carries it through global scratch and a global arrival counter (last CTA to arrive merges,
//     in CTA order; no CTA waits for another).  Results therefore do not depend on arrival
//     order, and no streaming warp executes a global fence or atomic.  A worker whose last head
//     runs past the CTA's range takes that piece first, which hides the global merge's latency
//     behind the rest of the streaming.
// Fused append (ssd_append_decode): the newest token's K/V rows are taken from the caller's
// k_new / v_new instead of the slab (the chunk that holds the token's ring slot is copied around
// that slot, and the two rows are copied into its place in the stage), and the worker that
// consumes that chunk writes the rows into the slab for later steps.  Nothing reads that slab slot
// during the launch, so no ordering is needed, and the per-layer append launch disappears.
// Every wait on an mbarrier is bounded: a warp that gives up raises a bit in the status word,
// waits (bounded again) for its other copies in flight and leaves.
#include <atomic>

#include "ssd_internal.cuh"
#include "ssd_device.cuh"

#ifndef SSD_DECODE_WARPS
#define SSD_DECODE_WARPS 8
#endif
#ifndef SSD_DECODE_STAGES
#define SSD_DECODE_STAGES 2
#endif
#ifndef SSD_DECODE_CHUNK
#define SSD_DECODE_CHUNK 16
#endif

namespace ssd {

namespace {

constexpr int kWarps = SSD_DECODE_WARPS;             // streaming workers per CTA
constexpr int kThreads = (kWarps + 1) * 32;          // plus one finisher warp
constexpr int kStages = SSD_DECODE_STAGES;
constexpr int kChunk = SSD_DECODE_CHUNK;             // slots per stage
constexpr int kGroups = 4;                           // 8-lane groups of a warp
constexpr int kPer = kChunk / kGroups;               // slots of a stage each group takes
constexpr int kU = kPer % 4 == 0 ? 4 : (kPer % 3 == 0 ? 3 : (kPer % 2 == 0 ? 2 : 1));   // slots a group folds in at a time
constexpr int kQBytes = kHeadDim * 2;
constexpr int kStageBytes = kChunk * kSlotBytes + kQBytes;
constexpr int kRingBytes = kWarps * kStages * kStageBytes;
constexpr int kBarBytes = (kWarps * kStages + 2) * 8;            // stage barriers, then the finisher's two
constexpr int kMailBoxes = kWarps * 2 + 2;                       // two partials per worker, two for the CTA
constexpr int kMailBytes = kMailBoxes * kPartialFloats * 4;
constexpr int kCountBytes = kWarps * 2 * 4;                      // arrival counter per (first worker, slot)
constexpr int kSmemBytes = kRingBytes + kBarBytes + kMailBytes + kCountBytes;

static_assert(kChunk % kGroups == 0 && kPer % kU == 0, "a stage is folded in groups of kGroups * kU slots");
static_assert(kSmemBytes <= 227 * 1024, "stage rings exceed the shared memory of an SM");
static_assert(kBarBytes % 16 == 0, "mailboxes are read as float4");
static_assert(2 * kWarps <= 32, "the finisher plans one possible post per lane");
static_assert((kWarps * kStages) % 2 == 0, "keeps the mailboxes 16-byte aligned");

// (m, l, acc4) <- (m, l, acc4) (+) (mj, lj, aj): four output dimensions of a partial
__device__ __forceinline__ void merge4(float& m, float& l, float4& acc, float mj, float lj, const float4& aj) {
  const float mn = fmaxf(m, mj);
  const float c1 = ex2(m - mn), c2 = ex2(mj - mn);
  l = l * c1 + lj * c2;
  acc.x = acc.x * c1 + aj.x * c2;
  acc.y = acc.y * c1 + aj.y * c2;
  acc.z = acc.z * c1 + aj.z * c2;
  acc.w = acc.w * c1 + aj.w * c2;
  m = mn;
}

__device__ __forceinline__ float dot16(const uint4& k0, const uint4& k1, const float2 (&q)[8]) {
  float2 a = make_float2(0.f, 0.f), b = make_float2(0.f, 0.f);
  a = __ffma2_rn(widen2(k0.x), q[0], a);
  b = __ffma2_rn(widen2(k1.x), q[4], b);
  a = __ffma2_rn(widen2(k0.y), q[1], a);
  b = __ffma2_rn(widen2(k1.y), q[5], b);
  a = __ffma2_rn(widen2(k0.z), q[2], a);
  b = __ffma2_rn(widen2(k1.z), q[6], b);
  a = __ffma2_rn(widen2(k0.w), q[3], a);
  b = __ffma2_rn(widen2(k1.w), q[7], b);
  return (a.x + a.y) + (b.x + b.y);
}

__device__ __forceinline__ void axpy16(float p, const uint4& v0, const uint4& v1, float2 (&acc)[8]) {
  const float2 pp = make_float2(p, p);
  acc[0] = __ffma2_rn(pp, widen2(v0.x), acc[0]);
  acc[1] = __ffma2_rn(pp, widen2(v0.y), acc[1]);
  acc[2] = __ffma2_rn(pp, widen2(v0.z), acc[2]);
  acc[3] = __ffma2_rn(pp, widen2(v0.w), acc[3]);
  acc[4] = __ffma2_rn(pp, widen2(v1.x), acc[4]);
  acc[5] = __ffma2_rn(pp, widen2(v1.y), acc[5]);
  acc[6] = __ffma2_rn(pp, widen2(v1.z), acc[6]);
  acc[7] = __ffma2_rn(pp, widen2(v1.w), acc[7]);
}

// The rows of a stage as one lane holds them: slot 4*u + grp, two 16-byte pieces of K and of V.
struct Rows {
  uint4 k0[kPer], k1[kPer], v0[kPer], v1[kPer];
};

// Pull the `n` slots of a stage out of shared memory so that the stage can be refilled before
// the arithmetic starts.
__device__ __forceinline__ void load_stage(const uint4* __restrict__ sb, int n, int grp, int l8, Rows& r) {
#pragma unroll
  for (int u = 0; u < kPer; ++u) {
    const int slot = kGroups * u + grp;
    const uint4* p = sb + slot * kSlotU4 + l8;
    if (slot < n) {
      r.k0[u] = p[0];
      r.k1[u] = p[8];
      r.v0[u] = p[16];
      r.v1[u] = p[24];
    } else {               // slots past n hold whatever an earlier chunk left there
      r.k0[u] = r.k1[u] = r.v0[u] = r.v1[u] = make_uint4(0, 0, 0, 0);
    }
  }
}

// Where the logits of a chunk go when the scores of semantic heads are being accumulated
// (Algorithm 2): row = the head's logit row (null: nothing to record), slot s of the chunk is valid
// slot i0 + s of the head; valid slots below `skip` are prompt slots (not scored) and those from
// `ring_from` on sit `ring_shift` entries further (unused static capacity in between).
struct LogitSink {
  float* row;
  int i0, skip, ring_from, ring_shift;
};

// Fold those slots into the running state of this lane's group.
__device__ __forceinline__ void fold_stage(const Rows& r, int n, int grp, int l8, const float2 (&q)[8], State& st,
                                           const LogitSink& sink) {
#pragma unroll
  for (int s = 0; s < kPer; s += kU) {
    if (kGroups * s >= n) break;
    float x[kU];
#pragma unroll
    for (int u = 0; u < kU; ++u) x[u] = dot16(r.k0[s + u], r.k1[s + u], q);
#pragma unroll
    for (int off = 4; off >= 1; off >>= 1) {
#pragma unroll
      for (int u = 0; u < kU; ++u) x[u] += __shfl_xor_sync(0xffffffffu, x[u], off);
    }
    if (sink.row != nullptr && l8 == 0) {
#pragma unroll
      for (int u = 0; u < kU; ++u) {
        const int slot = kGroups * (s + u) + grp;
        const int li = sink.i0 + slot;
        if (slot < n && li >= sink.skip) sink.row[li - sink.skip + (li >= sink.ring_from ? sink.ring_shift : 0)] = x[u];
      }
    }
    float mn = st.m;
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      if (kGroups * (s + u) + grp >= n) x[u] = kNegBig;
      mn = fmaxf(mn, x[u]);
    }
    const float corr = ex2(st.m - mn);
    float p[kU], psum = 0.f;
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      p[u] = kGroups * (s + u) + grp < n ? ex2(x[u] - mn) : 0.f;
      psum += p[u];
    }
    st.l = st.l * corr + psum;
    st.m = mn;
    const float2 cc = make_float2(corr, corr);
#pragma unroll
    for (int d = 0; d < 8; ++d) st.acc[d] = __fmul2_rn(st.acc[d], cc);
#pragma unroll
    for (int u = 0; u < kU; ++u) axpy16(p[u], r.v0[s + u], r.v1[s + u], st.acc);
  }
}

__device__ __forceinline__ uint32_t pack_bf16(float2 a, float inv) {
  __nv_bfloat162 t = __floats2bfloat162_rn(a.x * inv, a.y * inv);
  return *reinterpret_cast<uint32_t*>(&t);
}

// lanes 0..7 write the row: 16 bytes at dimension 8*l8 and 16 bytes at dimension 64 + 8*l8
__device__ __forceinline__ void write_out(__nv_bfloat16* out, const State& st, int l8) {
  const float inv = 1.f / st.l;
  uint4* o = reinterpret_cast<uint4*>(out);
  o[l8] = make_uint4(pack_bf16(st.acc[0], inv), pack_bf16(st.acc[1], inv), pack_bf16(st.acc[2], inv),
                     pack_bf16(st.acc[3], inv));
  o[8 + l8] = make_uint4(pack_bf16(st.acc[4], inv), pack_bf16(st.acc[5], inv), pack_bf16(st.acc[6], inv),
                         pack_bf16(st.acc[7], inv));
}

// all 32 lanes write the row, lane i the dimensions [4i, 4i + 4)
__device__ __forceinline__ void write_out4(__nv_bfloat16* out, float l, const float4& acc, int lane) {
  const float inv = 1.f / l;
  uint2 o;
  o.x = pack_bf16(make_float2(acc.x, acc.y), inv);
  o.y = pack_bf16(make_float2(acc.z, acc.w), inv);
  reinterpret_cast<uint2*>(out)[lane] = o;
}

// Which workers hold pieces of the head that spans logical slots [g0, g1), found by stepping from
// a worker `wk` known to hold one of them.
__device__ __forceinline__ void head_workers(const Split& sp, int wk, int g0, int g1, int& w_lo, int& w_hi) {
  w_lo = wk;
  while (w_lo > 0 && share_start(sp, w_lo) > g0) --w_lo;
  w_hi = wk;
  while (w_hi + 1 < sp.W && share_start(sp, w_hi + 1) < g1) ++w_hi;
}

// Fused append: valid-slot index, inside head h, of the token being appended (its ring slot holds
// stale bytes in the slab), and that slot's index from the head's first slot.
__device__ __forceinline__ void new_token_slot(const LayerView& v, int h, int new_j, int sem_slot, int& valid_idx, int& phys) {
  const HeadRec d = v.head[h];
  const int r = (d.w && sem_slot >= 0) ? sem_slot : new_j % d.z;   // a row buffer fills from its slot 0
  valid_idx = v.prompt_valid + (d.w ? v.static_valid : 0) + r;
  phys = v.L + d.y + r;
}

// Algorithm 2, score accumulation, deferred by one step: the weights of the layer's previous decode go into
// the scores at the start of the layer's next launch (nothing in that launch reads the scores), and the
// token being appended starts at zero.  Run by the finisher warp of every thread block, which share the
// pairs; entry c of a score row is static slot c or, from the static capacity on, buffer slot c - capacity.
__device__ void fold_scores(const DecodeParams& p, int lane) {
  const LayerView& v = p.view;
  const uint32_t FULL = 0xffffffffu;
  // This block's pairs are b, b + grid, ..; lane k looks at pair k, and the semantic ones are then taken four
  // at a time, all their loads issued before the first use: with HBM saturated by the streaming warps a
  // dependent trip to memory takes microseconds, so the trips must overlap; and the loop is kept free of
  // divisions, because this warp shares its scheduler with two streaming warps.
  constexpr int kFoldPairs = 4;
  const int n_pairs = v.n_seqs * v.H;
  const int n_mine = (n_pairs - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
  const int n_old = p.fold_pending ? p.fold_static + p.fold_buffered : 0;
  float* __restrict__ accp = p.fold_acc;
  const float* __restrict__ lgp = p.fold_logits;
  const float2* __restrict__ mlp = p.fold_ml;
  for (int k0 = 0; k0 < n_mine; k0 += 32) {
    const int my_pair = (int)blockIdx.x + (k0 + lane) * (int)gridDim.x;
    const bool sem = k0 + lane < n_mine && v.head[my_pair % v.H].w != 0;
    unsigned todo = __ballot_sync(FULL, sem);
    while (todo) {
      int pair[kFoldPairs], ycap[kFoldPairs], np = 0;
#pragma unroll
      for (int j = 0; j < kFoldPairs; ++j) {
        pair[j] = 0;
        ycap[j] = 0;
        if (todo) {
          const int src = __ffs(todo) - 1;
          todo &= todo - 1;
          pair[j] = __shfl_sync(FULL, my_pair, src);
          ycap[j] = v.head[pair[j] % v.H].y;
          np = j + 1;
        }
      }
      if (n_old > 0) {
        float2 ml[kFoldPairs];
#pragma unroll
        for (int j = 0; j < kFoldPairs; ++j) ml[j] = j < np ? mlp[pair[j]] : make_float2(0.f, 1.f);
        for (int i = lane; i < n_old; i += 32) {
          float a[kFoldPairs], x[kFoldPairs];
          uint32_t off[kFoldPairs];
#pragma unroll
          for (int j = 0; j < kFoldPairs; ++j) {
            // entry of the i-th scored token: static slot i, or buffer slot i - static behind the static capacity
            const int c = i < p.fold_static ? i : ycap[j] + (i - p.fold_static);
            off[j] = (uint32_t)pair[j] * (uint32_t)p.mr + (uint32_t)c;     // n_seqs * H * (M + R) < 2^31 (checked at create)
            if (j < np) {
              a[j] = accp[off[j]];
              x[j] = lgp[off[j]];
            }
          }
#pragma unroll
          for (int j = 0; j < kFoldPairs; ++j)
            if (j < np) accp[off[j]] = a[j] + ex2(x[j] - ml[j].x) / ml[j].y;
        }
      }
      if (p.sem_slot >= 0 && lane < np) {
        int pj = pair[0], yj = ycap[0];
#pragma unroll
        for (int j = 1; j < kFoldPairs; ++j)
          if (lane == j) { pj = pair[j]; yj = ycap[j]; }
        accp[(size_t)pj * p.mr + yj + p.sem_slot] = 0.f;       // the token being appended starts at zero
      }
    }
  }
}

// The finisher warp of a CTA carries the (at most two) heads that cross the CTA's own range
// through global memory: it waits for the CTA's merged partial of such a head (left in a shared-
// memory mailbox by the worker that completed it), stores it in global scratch, counts arrivals
// per head with an atomic (it never waits for another CTA) and, where this CTA was the last to
// arrive, merges the CTAs' partials in CTA order.  All global fences and atomics of the launch
// are issued here, off the streaming warps' path.  Lane i holds output dimensions [4i, 4i + 4).
__device__ void finisher(const DecodeParams& p, const unsigned char* smem, int lane) {
  const LayerView& v = p.view;
  const Split& sp = p.split;
  const uint32_t FULL = 0xffffffffu;
  const uint32_t cta_bar0 = smem_u32(smem + kRingBytes) + kWarps * kStages * 8;
  const float* cta_mail = reinterpret_cast<const float*>(smem + kRingBytes + kBarBytes) +
                          (size_t)kWarps * 2 * kPartialFloats;
  const int lo_c = (int)blockIdx.x * kWarps;
  const int hi_c = (lo_c + kWarps < sp.W ? lo_c + kWarps : sp.W) - 1;
  const int r_begin = share_start(sp, lo_c), r_end = share_start(sp, hi_c + 1);   // the CTA's range

  // lane 0: the head that covers the range's first slot, if it began earlier; lane 1: the head
  // that covers its last slot, if it runs on (and is not the same head)
  int r_pair = -1, r_clo = 0, r_chi = 0;
  if (lane < 2 && r_begin < r_end) {
    Walk t;
    const int g = lane == 0 ? r_begin : r_end - 1;
    walk_init(t, v, g, r_end);
    const int g0 = g - t.i, g1 = g0 + t.vh;
    const bool crosses = lane == 0 ? g0 < r_begin : (g1 > r_end && g0 >= r_begin);
    if (crosses) {
      int w_lo, w_hi;
      head_workers(sp, lane == 0 ? lo_c : hi_c, g0, g1, w_lo, w_hi);
      r_pair = t.seq * v.H + t.head;
      r_clo = w_lo / kWarps;
      r_chi = w_hi / kWarps;
    }
  }
  unsigned heads = __ballot_sync(FULL, r_pair >= 0);
  if (!heads && p.fold_acc == nullptr) return;
  pdl_wait_predecessor();                // the scratch below may still be in use by the previous launch
  pdl_allow_successor();
  if (p.fold_acc != nullptr) fold_scores(p, lane);
  if (!heads) return;
  for (unsigned h = heads; h; h &= h - 1) {
    const int slot = __ffs(h) - 1;       // 0: began in an earlier CTA, 1: begins here and runs on
    if (!mbar_wait(cta_bar0 + 8 * slot, 0)) {
      if (lane == 0) atomicOr(p.status, 1u);
      return;
    }
    const float4* src = reinterpret_cast<const float4*>(cta_mail + (size_t)slot * kPartialFloats);
    float4* dst = reinterpret_cast<float4*>(p.partial + ((size_t)blockIdx.x * 2 + slot) * kPartialFloats);
    dst[1 + lane] = src[1 + lane];
    if (lane == 0) dst[0] = src[0];
  }
  __threadfence();                       // the partials above, before the arrivals below
  bool last_in = false;
  if (r_pair >= 0) last_in = atomicAdd(p.counters + r_pair, 1u) == (uint32_t)(r_chi - r_clo);
  unsigned todo = __ballot_sync(FULL, last_in);
  if (todo) __threadfence();
  while (todo) {
    const int src = __ffs(todo) - 1;
    todo &= todo - 1;
    const int pair = __shfl_sync(FULL, r_pair, src);
    const int c_lo = __shfl_sync(FULL, r_clo, src), c_hi = __shfl_sync(FULL, r_chi, src);
    float m = kNegBig, l = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int c = c_lo; c <= c_hi; ++c) {
      const float* G = p.partial + ((size_t)c * 2 + (c > c_lo ? 0 : 1)) * kPartialFloats;
      merge4(m, l, acc, __ldcg(G), __ldcg(G + 1), __ldcg(reinterpret_cast<const float4*>(G + 4) + lane));
    }
    write_out4(p.out + (size_t)pair * kHeadDim, l, acc, lane);
    if (p.ml != nullptr && lane == 0) p.ml[pair] = make_float2(m, l);
    if (lane == 0) p.counters[pair] = 0u;
  }
}

__global__ void __launch_bounds__(kThreads, 1) ssd_decode_kernel(const __grid_constant__ DecodeParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  const LayerView& v = p.view;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int grp = lane >> 3, l8 = lane & 7;

  const uint32_t bar0 = smem_u32(smem + kRingBytes) + (uint32_t)warp * kStages * 8;
  const uint32_t cta_bar0 = smem_u32(smem + kRingBytes) + kWarps * kStages * 8;
  float* mail = reinterpret_cast<float*>(smem + kRingBytes + kBarBytes);
  int* arrivals = reinterpret_cast<int*>(smem + kRingBytes + kBarBytes + kMailBytes);
  if (lane == 0) {
    if (warp < kWarps) {
#pragma unroll
      for (int s = 0; s < kStages; ++s) mbar_init(bar0 + 8 * s, 1);
      arrivals[2 * warp] = 0;
      arrivals[2 * warp + 1] = 0;
    } else {
      mbar_init(cta_bar0, 1);
      mbar_init(cta_bar0 + 8, 1);
    }
    mbar_init_fence();
  }
  __syncthreads();   // the only CTA-wide barrier: counters and barriers exist before anyone uses them

  if (warp == kWarps) {
    finisher(p, smem, lane);
    return;
  }
  const int wk = (int)blockIdx.x * kWarps + warp;
  if (wk >= p.split.W) return;
  const int g_begin = share_start(p.split, wk), g_end = share_start(p.split, wk + 1);
  if (g_begin >= g_end) return;
  // If the head at the end of the share runs past this CTA's range, its merge goes through global
  // memory: take that piece first ([g_tail, g_end), then [g_begin, g_tail)) so that the merge's
  // latency is hidden behind the rest of the streaming.  Otherwise stream order (g_tail == g_end).
  int g_tail = g_end;
  {
    const int w_next = ((int)blockIdx.x + 1) * kWarps < p.split.W ? ((int)blockIdx.x + 1) * kWarps : p.split.W;
    const int cta_end = share_start(p.split, w_next);
    if (cta_end - g_end < v.max_vh) {
      Walk t;
      walk_init(t, v, g_end - 1, g_end);
      const int head_start = g_end - 1 - t.i;
      if (head_start + t.vh > cta_end) g_tail = head_start > g_begin ? head_start : g_begin;
    }
  }
  const bool two_parts = g_begin < g_tail && g_tail < g_end;
  auto advance = [&](Walk& w, int n) {
    walk_advance(w, v, n);
    if (two_parts && w.g == g_end && w.g_end == g_end) walk_init(w, v, g_begin, g_tail);
  };

  unsigned char* ring = smem + (size_t)warp * kStages * kStageBytes;
  const uint32_t ring_s = smem_u32(ring);
  const int lo_c = (int)blockIdx.x * kWarps;
  const int hi_c = (lo_c + kWarps < p.split.W ? lo_c + kWarps : p.split.W) - 1;

  Walk prod;
  walk_init(prod, v, two_parts ? g_tail : g_begin, g_end);
  Walk cons = prod;
  int ahead = 0;   // chunks issued and not yet consumed

  // Lane 0 starts copies of the chunk at a walk position into a stage, in two steps: planning (everything that
  // needs the layout tables: where the head starts, where the newest token sits, the rows of the caller's
  // inputs) and firing (fence, byte count, the copies).  The main loop plans the next chunk while it waits for
  // the current one's data, so that between "the stage is free" and "its refill is on its way" only the firing
  // remains.  what & 1: the slab part (and the barrier's byte count for the whole chunk); what & 2: the caller's
  // inputs that travel with the chunk (the head's query row with its first chunk, the newest token's rows in
  // place of its slot).
  struct Plan {
    const unsigned char* hbase;   // the head's first slot
    size_t row;                   // byte offset of the head's row in q, k_new, v_new
    int head, i, n;               // valid slots [i, i + n) of the head
    int fresh;                    // valid-slot index of the newest token in this head (-1: none)
    bool begin;                   // the chunk carries the head's query row
  };
  int pf_key = -1, pf_fresh = -1, pf_phys = 0;     // producer side: newest token's slot in the current head
  auto plan_chunk = [&](const Walk& w, Plan& pl) {
    pl.n = walk_chunk(w, kChunk);
    pl.i = w.i;
    pl.head = w.head;
    pl.begin = w.i == 0 || w.g == g_begin;
    if (lane != 0) return;
    pl.hbase = reinterpret_cast<const unsigned char*>(p.slab) + ((size_t)w.seq * v.seq_slots + v.head[w.head].x) * kSlotBytes;
    if (p.new_j >= 0 && pf_key != w.seq * v.H + w.head) {      // once per head, not per chunk
      pf_key = w.seq * v.H + w.head;
      new_token_slot(v, w.head, p.new_j, p.sem_slot, pf_fresh, pf_phys);
    }
    pl.fresh = pf_fresh;
    pl.row = ((size_t)w.seq * v.H + w.head) * kQBytes;
  };
  auto fire_chunk = [&](const Plan& pl, int stage, int what) {
    if (lane != 0) return;
    const uint32_t dst = ring_s + (uint32_t)stage * kStageBytes, bar = bar0 + 8 * stage;
    const int fresh = pl.fresh, n = pl.n;
    const bool has_fresh = fresh >= pl.i && fresh < pl.i + n;
    if (what & 1) {
      // order the warp's reads of this stage (made visible to this lane by __syncwarp) before
      // the asynchronous writes that follow
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      mbar_expect_tx(bar, (uint32_t)(n * kSlotBytes + (pl.begin ? kQBytes : 0)));
      // valid slots [a, a + len) of the head into the stage from slot `at` on
      auto copy_range = [&](int a, int len, int at) {
        if (len <= 0) return;
        if (v.contig) {
          bulk_g2s(dst + (uint32_t)at * kSlotBytes, pl.hbase + (size_t)a * kSlotBytes, (uint32_t)len * kSlotBytes, bar);
        } else {
          chunk_runs(v, pl.head, a, len, [&](int src, int d, int l) {
            bulk_g2s(dst + (uint32_t)(at + d) * kSlotBytes, pl.hbase + (size_t)src * kSlotBytes, (uint32_t)l * kSlotBytes, bar);
          });
        }
      };
      if (has_fresh) {                   // the slab is copied around the newest token's slot
        copy_range(pl.i, fresh - pl.i, 0);
        copy_range(fresh + 1, pl.i + n - fresh - 1, fresh + 1 - pl.i);
      } else {
        copy_range(pl.i, n, 0);
      }
    }
    if (what & 2) {
      if (has_fresh) {
        bulk_g2s(dst + (uint32_t)(fresh - pl.i) * kSlotBytes, p.k_new + pl.row, kQBytes, bar);
        bulk_g2s(dst + (uint32_t)(fresh - pl.i) * kSlotBytes + kQBytes, p.v_new + pl.row, kQBytes, bar);
      }
      if (pl.begin) bulk_g2s(dst + kChunk * kSlotBytes, reinterpret_cast<const unsigned char*>(p.q) + pl.row, kQBytes, bar);
    }
  };
  auto copy_chunk = [&](const Walk& w, int stage, int what) {
    Plan pl;
    plan_chunk(w, pl);
    fire_chunk(pl, stage, what);
  };

  // Prologue.  Everything above read only the launch parameters.  The slab holds nothing that the
  // preceding launch writes when that launch worked on another layer (p.early), so the first
  // chunks' slab copies may start while it is still running; the caller's inputs (q, new rows) and
  // every write wait until it has completed.
  if (!p.early) {
    pdl_wait_predecessor();
    pdl_allow_successor();
  }
  const Walk prod0 = prod;
  int n_pro = 0;
#pragma unroll 1
  for (; n_pro < kStages && prod.g < prod.g_end; ++n_pro) {
    copy_chunk(prod, n_pro, p.early ? 1 : 3);
    advance(prod, walk_chunk(prod, kChunk));
    ++ahead;
  }
  if (p.early) {
    pdl_wait_predecessor();
    pdl_allow_successor();
    Walk redo = prod0;
#pragma unroll 1
    for (int s = 0; s < n_pro; ++s) {
      copy_chunk(redo, s, 2);
      advance(redo, walk_chunk(redo, kChunk));
    }
  }

  int stage = 0;
  uint32_t parity = 0;
  bool begin = true, leading = true;
  int piece_i0 = 0;
  float2 q[8];
  State st;
  LogitSink sink = {nullptr, 0, 0, 0, 0};
  int fresh = -1, fresh_phys = 0;                   // consumer side: newest token's slot in the current head

#pragma unroll 1
  while (cons.g < cons.g_end) {
    const int n = walk_chunk(cons, kChunk);
    Plan next;                                     // the chunk that will refill this stage, planned while its data is awaited
    const bool more = prod.g < prod.g_end;
    if (more) plan_chunk(prod, next);
    if (!mbar_wait(bar0 + 8 * stage, parity)) {
      // give up: flag it, let the copies still in flight land (bounded), and leave
      if (lane == 0) atomicOr(p.status, 1u);
      for (int k = 0; k < ahead; ++k) {
        mbar_wait(bar0 + 8 * stage, parity);
        if (++stage == kStages) { stage = 0; parity ^= 1u; }
      }
      return;
    }
    const uint4* sb = reinterpret_cast<const uint4*>(ring + (size_t)stage * kStageBytes);
    if (begin) {
      const uint4 qa = sb[kChunk * kSlotU4 + l8], qb = sb[kChunk * kSlotU4 + 8 + l8];
      const float2 sc = make_float2(p.scale_log2, p.scale_log2);
      q[0] = __fmul2_rn(widen2(qa.x), sc); q[1] = __fmul2_rn(widen2(qa.y), sc);
      q[2] = __fmul2_rn(widen2(qa.z), sc); q[3] = __fmul2_rn(widen2(qa.w), sc);
      q[4] = __fmul2_rn(widen2(qb.x), sc); q[5] = __fmul2_rn(widen2(qb.y), sc);
      q[6] = __fmul2_rn(widen2(qb.z), sc); q[7] = __fmul2_rn(widen2(qb.w), sc);
      state_init(st);
      piece_i0 = cons.i;
      leading = cons.g == g_begin;      // the piece that holds the share's first slot
      begin = false;
      const HeadRec d = v.head[cons.head];
      sink.row = (p.logits != nullptr && d.w) ? p.logits + ((size_t)cons.seq * v.H + cons.head) * p.mr : nullptr;
      sink.skip = v.prompt_valid;
      sink.ring_from = v.prompt_valid + v.static_valid;
      sink.ring_shift = d.y - v.static_valid;
      if (p.new_j >= 0) new_token_slot(v, cons.head, p.new_j, p.sem_slot, fresh, fresh_phys);
    }
    sink.i0 = cons.i;
    Rows rows;
    load_stage(sb, n, grp, l8, rows);
    if (p.new_j >= 0) {
      // fused append: the chunk that carries the newest token also stores it in the slab
      const int s_new = fresh - cons.i;
      if (s_new >= 0 && s_new < n) {
        uint4* dstrow = const_cast<uint4*>(p.slab) +
                        ((size_t)cons.seq * v.seq_slots + v.head[cons.head].x + fresh_phys) * kSlotU4;
        dstrow[lane] = sb[s_new * kSlotU4 + lane];
      }
    }
    __syncwarp();          // every lane has its rows in registers: the stage may be refilled
    --ahead;
    if (more) {
      fire_chunk(next, stage, 3);
      advance(prod, next.n);
      ++ahead;
    }
    fold_stage(rows, n, grp, l8, q, st, sink);

    const int i1 = cons.i + n;
    if (i1 == cons.vh || cons.g + n == cons.g_end) {
      // end of this worker's piece of the head: merge the four groups (lanes l, l^8, l^16, l^24
      // hold the same 16 output dims), then write the output, or post a partial to the finisher
      State tot = st;
      state_merge_lane(tot, 8);
      state_merge_lane(tot, 16);
      if (piece_i0 == 0 && i1 == cons.vh) {
        if (grp == 0) write_out(p.out + ((size_t)cons.seq * v.H + cons.head) * kHeadDim, tot, l8);
        if (p.ml != nullptr && lane == 0) p.ml[(size_t)cons.seq * v.H + cons.head] = make_float2(tot.m, tot.l);
      } else {
        // post the partial; the worker that posts a head's last piece in this CTA merges them
        float* P = mail + (size_t)(2 * warp + (leading ? 0 : 1)) * kPartialFloats;
        if (lane == 0) {
          P[0] = tot.m;
          P[1] = tot.l;
        }
        if (grp == 0) {
          float4* lo = reinterpret_cast<float4*>(P + 4 + 8 * l8);
          float4* hi = reinterpret_cast<float4*>(P + 4 + 64 + 8 * l8);
          lo[0] = make_float4(tot.acc[0].x, tot.acc[0].y, tot.acc[1].x, tot.acc[1].y);
          lo[1] = make_float4(tot.acc[2].x, tot.acc[2].y, tot.acc[3].x, tot.acc[3].y);
          hi[0] = make_float4(tot.acc[4].x, tot.acc[4].y, tot.acc[5].x, tot.acc[5].y);
          hi[1] = make_float4(tot.acc[6].x, tot.acc[6].y, tot.acc[7].x, tot.acc[7].y);
        }
        const int g0 = cons.g - cons.i, g1 = g0 + cons.vh;    // the whole head in the stream
        int w_lo, w_hi;
        head_workers(p.split, wk, g0, g1, w_lo, w_hi);
        const int f = w_lo > lo_c ? w_lo : lo_c, e = w_hi < hi_c ? w_hi : hi_c;   // holders in this CTA
        // worker j holds the head in its slot 0 (leading piece), unless the head starts inside j's share
        const int locut = share_start(p.split, w_lo) < g0 ? 1 : 0;
        const int f_box = (f - lo_c) * 2 + ((f == w_lo && locut) ? 1 : 0);
        __syncwarp();
        int old = 0;
        if (lane == 0) {
          __threadfence_block();
          old = atomicAdd(arrivals + f_box, 1);
        }
        old = __shfl_sync(0xffffffffu, old, 0);
        if (old == e - f) {
          __threadfence_block();
          float m = kNegBig, l = 0.f;
          float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
          for (int j = f; j <= e; ++j) {
            const float* Pj = mail + (size_t)((j - lo_c) * 2 + ((j == w_lo && locut) ? 1 : 0)) * kPartialFloats;
            merge4(m, l, acc, Pj[0], Pj[1], reinterpret_cast<const float4*>(Pj + 4)[lane]);
          }
          if (w_lo >= lo_c && w_hi <= hi_c) {              // the whole head lies inside this CTA
            write_out4(p.out + ((size_t)cons.seq * v.H + cons.head) * kHeadDim, l, acc, lane);
            if (p.ml != nullptr && lane == 0) p.ml[(size_t)cons.seq * v.H + cons.head] = make_float2(m, l);
          } else {                                         // hand the CTA's partial to the finisher
            const int slot = w_lo < lo_c ? 0 : 1;
            float* C = mail + (size_t)(2 * kWarps + slot) * kPartialFloats;
            if (lane == 0) {
              C[0] = m;
              C[1] = l;
            }
            reinterpret_cast<float4*>(C + 4)[lane] = acc;
            __syncwarp();
            if (lane == 0) mbar_arrive(cta_bar0 + 8 * slot);   // releases the writes above
          }
        }
      }
      begin = true;
    }
    advance(cons, n);
    if (++stage == kStages) { stage = 0; parity ^= 1u; }
  }
}

// ------------------------------------------------------------------ a whole step in one launch
// Fused append + decode of every layer.  With all layers in one launch there are tens of thousands
// of heads to go round, so no head needs to be cut: the unit of work is one whole head of one
// (layer, sequence), units are handed out in stream order from a global counter to whichever warp
// asks next (warps on slower SMs simply take fewer), and a head is finished in the registers of the
// warp that streamed it.  No partials, no mailboxes, no finisher, no barrier after start-up.  A
// warp's copy pipeline runs on across unit boundaries: the next unit is claimed while the current
// one streams, and its first chunks are in flight before the current head's arithmetic ends.
struct Unit {
  const unsigned char* hbase;   // the head's first slot
  size_t row;                   // byte offset of the head's row in q, k_new, v_new (and out)
  int vh;                       // slots that hold a token
  int pv, sv;                   // of which prompt slots and static slots (the rest is the ring)
  int y;                        // static capacity (slots between the prompt and the ring)
  int fresh;                    // valid-slot index of the token being appended
  int phys;                     // and its slot counted from the head's first slot
  int contig;                   // the valid slots are one physical run
  int u;                        // the unit's number
  int scored;                   // 1: a semantic head whose attention scores are accumulated (Algorithm 2)
};

__device__ __forceinline__ void unit_load(const DecodeLayersParams& p, int u, Unit& U) {
  const int pairs = p.n_seqs * p.H;
  const int layer = u / pairs, pair = u - layer * pairs;
  const int seq = pair / p.H, head = pair - seq * p.H;
  const LayerState& ls = p.layer[layer];
  const HeadDesc d = __ldg(ls.desc + head);
  U.u = u;
  U.scored = (p.acc != nullptr && d.w) ? 1 : 0;
  const int held = U.scored ? ls.t_sem : ls.t_img;          // tokens the ring holds
  const int r = U.scored ? ls.sem_slot : ls.new_j % d.z;    // ring slot of the token being appended
  U.pv = ls.prompt_valid;
  U.sv = d.w ? ls.static_valid : 0;
  U.y = d.y;
  U.vh = U.pv + U.sv + (held < d.z ? held : d.z);
  U.fresh = U.pv + U.sv + r;
  U.phys = p.L + d.y + r;
  U.contig = (U.pv == p.L && U.sv == d.y) ? 1 : 0;
  U.hbase = reinterpret_cast<const unsigned char*>(p.slab) +
            ((size_t)ls.first_slot + (size_t)seq * ls.seq_slots + d.x) * kSlotBytes;
  U.row = ((size_t)layer * pairs + pair) * kQBytes;
}

constexpr int kLayersSmemBytes = kRingBytes + kWarps * kStages * 8 + kWarps * 4 * 4;

// kEvict: Algorithm 1 taken literally (a row buffer of one token, re-selected in the same launch).
template <bool kEvict>
__global__ void __launch_bounds__(kWarps * 32, 1) ssd_decode_layers_kernel(const __grid_constant__ DecodeLayersParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int grp = lane >> 3, l8 = lane & 7;
  const uint32_t FULL = 0xffffffffu;
  unsigned char* ring = smem + (size_t)warp * kStages * kStageBytes;
  const uint32_t ring_s = smem_u32(ring);
  const uint32_t bar0 = smem_u32(smem + kRingBytes) + (uint32_t)warp * kStages * 8;
  volatile int* fifo = reinterpret_cast<volatile int*>(smem + kRingBytes + kWarps * kStages * 8) + warp * 4;
  // row-buffer mode: the logits of the head being streamed, entry e = static slot e or, from the
  // static capacity on, buffer slot e - capacity (the layout of the score rows)
  const int mrp = (p.mr + 3) & ~3;
  float* lgbuf = reinterpret_cast<float*>(smem + kLayersSmemBytes) + (size_t)warp * mrp * (kEvict ? 3 : 1);
  float* accbuf = lgbuf + mrp;                         // kEvict: the head's score row ...
  int* idxbuf = reinterpret_cast<int*>(accbuf + mrp);  // ... and the image indices of its static slots
  if (lane == 0) {
#pragma unroll
    for (int s = 0; s < kStages; ++s) mbar_init(bar0 + 8 * s, 1);
    mbar_init_fence();
  }
  __syncwarp();
  const int n_units = p.n_layers * p.n_seqs * p.H;

  // unit ids come from the counter; lane 0 asks for the next one long before it is needed
  int raw_next = 0;
  auto ask = [&]() {
    if (lane == 0) raw_next = (int)atomicAdd(p.work, 1u);
  };
  ask();
  int u = __shfl_sync(FULL, raw_next, 0);
  if (u >= n_units) return;
  ask();

  Unit PU, CU;                 // the producer's and the consumer's current head
  int pi = 0, ci = 0;          // and their positions in it
  int produced = 0, consumed = 0, ahead = 0;
  bool feeding = true;
  unit_load(p, u, PU);
  if (lane == 0) fifo[0] = u;
  produced = 1;
  __syncwarp();

  // Lane 0 starts the copies of the producer's next chunk into `stage`; every lane advances.
  auto issue = [&](int stage) {
    const int n = PU.vh - pi < kChunk ? PU.vh - pi : kChunk;
    if (lane == 0) {
      const bool begin = pi == 0;
      const uint32_t dst = ring_s + (uint32_t)stage * kStageBytes, bar = bar0 + 8 * stage;
      const bool has_fresh = PU.fresh >= pi && PU.fresh < pi + n;
      // order the warp's reads of this stage (made visible to this lane by __syncwarp) before
      // the asynchronous writes that follow
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      mbar_expect_tx(bar, (uint32_t)(n * kSlotBytes + (begin ? kQBytes : 0)));
      // valid slots [a, a + len) of the head into the stage from slot `at` on
      auto copy_range = [&](int a, int len, int at) {
        if (len <= 0) return;
        if (PU.contig) {
          bulk_g2s(dst + (uint32_t)at * kSlotBytes, PU.hbase + (size_t)a * kSlotBytes, (uint32_t)len * kSlotBytes, bar);
          return;
        }
        const int l0[3] = {0, PU.pv, PU.pv + PU.sv};          // logical start of each run
        const int l1[3] = {PU.pv, PU.pv + PU.sv, PU.vh};      // and end
        const int p0[3] = {0, p.L, p.L + PU.y};               // physical start
#pragma unroll
        for (int r = 0; r < 3; ++r) {
          const int lo = a > l0[r] ? a : l0[r], hi = a + len < l1[r] ? a + len : l1[r];
          if (hi > lo)
            bulk_g2s(dst + (uint32_t)(at + lo - a) * kSlotBytes, PU.hbase + (size_t)(p0[r] + lo - l0[r]) * kSlotBytes,
                     (uint32_t)(hi - lo) * kSlotBytes, bar);
        }
      };
      if (has_fresh) {                   // the slab is copied around the newest token's slot
        copy_range(pi, PU.fresh - pi, 0);
        copy_range(PU.fresh + 1, pi + n - PU.fresh - 1, PU.fresh + 1 - pi);
        bulk_g2s(dst + (uint32_t)(PU.fresh - pi) * kSlotBytes, p.k_new + PU.row, kQBytes, bar);
        bulk_g2s(dst + (uint32_t)(PU.fresh - pi) * kSlotBytes + kQBytes, p.v_new + PU.row, kQBytes, bar);
      } else {
        copy_range(pi, n, 0);
      }
      if (begin) bulk_g2s(dst + kChunk * kSlotBytes, p.q + PU.row, kQBytes, bar);
    }
    pi += n;
    ++ahead;
    if (pi == PU.vh) {                   // on to the unit asked for earlier, and ask for the one after
      const int nu = __shfl_sync(FULL, raw_next, 0);
      if (nu < n_units) {
        ask();
        unit_load(p, nu, PU);
        pi = 0;
        if (lane == 0) fifo[produced & 3] = nu;
        ++produced;
        __syncwarp();
      } else {
        feeding = false;
      }
    }
  };

#pragma unroll 1
  for (int s = 0; s < kStages && feeding; ++s) issue(s);

  int stage = 0;
  uint32_t parity = 0;
  float2 q[8];
  State st;
  LogitSink sink = {nullptr, 0, 0, 0, 0};
  bool begin = true;

#pragma unroll 1
  for (;;) {
    if (begin) {
      if (consumed == produced) break;
      unit_load(p, fifo[consumed & 3], CU);
      ++consumed;
      ci = 0;
    }
    const int n = CU.vh - ci < kChunk ? CU.vh - ci : kChunk;
    if (!mbar_wait(bar0 + 8 * stage, parity)) {
      // give up: flag it, let the copies still in flight land (bounded), and leave
      if (lane == 0) atomicOr(p.status, 1u);
      for (int k = 0; k < ahead; ++k) {
        mbar_wait(bar0 + 8 * stage, parity);
        if (++stage == kStages) { stage = 0; parity ^= 1u; }
      }
      return;
    }
    const uint4* sb = reinterpret_cast<const uint4*>(ring + (size_t)stage * kStageBytes);
    if (begin) {
      const uint4 qa = sb[kChunk * kSlotU4 + l8], qb = sb[kChunk * kSlotU4 + 8 + l8];
      const float2 sc = make_float2(p.scale_log2, p.scale_log2);
      q[0] = __fmul2_rn(widen2(qa.x), sc); q[1] = __fmul2_rn(widen2(qa.y), sc);
      q[2] = __fmul2_rn(widen2(qa.z), sc); q[3] = __fmul2_rn(widen2(qa.w), sc);
      q[4] = __fmul2_rn(widen2(qb.x), sc); q[5] = __fmul2_rn(widen2(qb.y), sc);
      q[6] = __fmul2_rn(widen2(qb.z), sc); q[7] = __fmul2_rn(widen2(qb.w), sc);
      state_init(st);
      begin = false;
      sink.row = CU.scored ? lgbuf : nullptr;
      sink.skip = CU.pv;
      sink.ring_from = CU.pv + CU.sv;
      sink.ring_shift = CU.y - CU.sv;
      if (kEvict && CU.scored) {
        // the head's scores and static positions are wanted when its last chunk is done: start them
        // towards shared memory now (4-byte asynchronous copies; nothing waits for them here)
        const int pairs = p.n_seqs * p.H, layer = CU.u / pairs;
        const size_t pr = (size_t)layer * pairs + (CU.u - layer * pairs);
        const float* acc = p.acc + pr * p.mr;
        const int32_t* idx = p.static_idx + pr * (p.M > 0 ? p.M : 1);
        for (int i = lane; i < CU.sv; i += 32) {
          asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(accbuf + i)), "l"(acc + i) : "memory");
          asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(idxbuf + i)), "l"(idx + i) : "memory");
        }
      }
    }
    sink.i0 = ci;
    Rows rows;
    load_stage(sb, n, grp, l8, rows);
    {
      // the chunk that carries the newest token also stores it in the slab
      const int s_new = CU.fresh - ci;
      if (s_new >= 0 && s_new < n) {
        uint4* dstrow = reinterpret_cast<uint4*>(const_cast<unsigned char*>(CU.hbase)) + (size_t)CU.phys * kSlotU4;
        dstrow[lane] = sb[s_new * kSlotU4 + lane];
      }
    }
    __syncwarp();          // every lane has its rows in registers: the stage may be refilled
    --ahead;
    if (feeding) issue(stage);
    fold_stage(rows, n, grp, l8, q, st, sink);
    ci += n;
    if (ci == CU.vh) {
      // the head is complete: merge the four groups and write the output row
      State tot = st;
      state_merge_lane(tot, 8);
      state_merge_lane(tot, 16);
      if (grp == 0) write_out(reinterpret_cast<__nv_bfloat16*>(reinterpret_cast<unsigned char*>(p.out) + CU.row), tot, l8);
      if (kEvict && CU.scored) {
        // Algorithm 1, one step: add the step's attention weights to the scores, then keep the M best
        // of the static tokens and the token just appended (lowest score leaves; among equal scores
        // the highest position, so the new token loses ties).  The new token's rows were stored in the
        // head's one-slot buffer above by these very lanes; if it stays, they copy it into the static
        // slot that is free or freed.  Nothing of this head is in flight any more: all its chunks are
        // consumed.
        asm volatile("cp.async.wait_all;" ::: "memory");
        __syncwarp();                    // scores, positions and logits in shared memory, for every lane
        const int pairs = p.n_seqs * p.H, layer = CU.u / pairs;
        const size_t pr = (size_t)layer * pairs + (CU.u - layer * pairs);
        float* acc = p.acc + pr * p.mr;
        int32_t* idx = p.static_idx + pr * (p.M > 0 ? p.M : 1);
        const float inv = 1.f / tot.l;
        const int sv = CU.sv;
        float worst = 3.0e38f;
        int worst_pos = -1, worst_e = -1;
        for (int i = lane; i < sv; i += 32) {
          const float sc = accbuf[i] + ex2(lgbuf[i] - tot.m) * inv;
          accbuf[i] = sc;
          const int pos = idxbuf[i];
          if (sc < worst || (sc == worst && pos > worst_pos)) { worst = sc; worst_pos = pos; worst_e = i; }
        }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
          const float w2 = __shfl_xor_sync(FULL, worst, off);
          const int p2 = __shfl_xor_sync(FULL, worst_pos, off), e2 = __shfl_xor_sync(FULL, worst_e, off);
          if (w2 < worst || (w2 == worst && p2 > worst_pos)) { worst = w2; worst_pos = p2; worst_e = e2; }
        }
        const float w_new = ex2(lgbuf[CU.phys - p.L] - tot.m) * inv;   // the new token's score starts here
        int dest = -1;                                                 // static slot the new token takes
        if (sv < p.M) dest = sv;
        else if (sv > 0 && !(w_new <= worst)) dest = worst_e;
        for (int i = lane; i < sv; i += 32)
          if (i != dest) acc[i] = accbuf[i];
        if (dest >= 0) {
          if (lane == 0) {
            acc[dest] = w_new;
            idx[dest] = p.layer[layer].new_j;
          }
          uint4* hb = reinterpret_cast<uint4*>(const_cast<unsigned char*>(CU.hbase));
          hb[(size_t)(p.L + dest) * kSlotU4 + lane] = hb[(size_t)CU.phys * kSlotU4 + lane];
        }
        __syncwarp();                    // before the next head's copies and logits reuse the buffers
      } else if (CU.scored) {
        // Algorithm 2, post-processing (score accumulation): this warp saw the whole head, so the
        // normalised weights go straight into the head's score row (which no other warp touches;
        // additions without a return value, so nothing waits for them).  The token appended in this
        // step starts its score here.
        __syncwarp();                    // the logits written by the group leaders, for every lane
        const int pairs = p.n_seqs * p.H, layer = CU.u / pairs;
        float* acc = p.acc + ((size_t)layer * pairs + (CU.u - layer * pairs)) * p.mr;
        const float inv = 1.f / tot.l;
        const int n_scored = CU.vh - CU.pv, e_new = CU.phys - p.L;     // entries that hold a token; the new one
        for (int i = lane; i < n_scored; i += 32) {
          const int e = i < CU.sv ? i : CU.y + (i - CU.sv);
          const float w = ex2(lgbuf[e] - tot.m) * inv;
          if (e == e_new) acc[e] = w;
          else atomicAdd(acc + e, w);
        }
        __syncwarp();                    // before the next head's logits overwrite the buffer
      }
      begin = true;
    }
    if (++stage == kStages) { stage = 0; parity ^= 1u; }
  }
}

// acc += exp2(logit - max) / sum over the entries that held a token at the layer's last decode
__global__ void __launch_bounds__(256) ssd_fold_pending_kernel(float* acc, const float* logits, const float2* ml,
                                                               const HeadDesc* desc, int n_pairs, int H, int mr,
                                                               int static_valid, int buffered) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= n_pairs) return;
  const HeadDesc d = desc[warp % H];
  if (!d.w) return;
  float* a = acc + (size_t)warp * mr;
  const float* lg = logits + (size_t)warp * mr;
  const float2 s = ml[warp];
  const float inv = 1.f / s.y;
  for (int i = lane; i < static_valid + buffered; i += 32) {
    const int c = i < static_valid ? i : d.y + (i - static_valid);
    a[c] += ex2(lg[c] - s.x) * inv;
  }
}

__global__ void __launch_bounds__(256) ssd_append_kernel(const AppendParams p) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  pdl_wait_predecessor();
  pdl_allow_successor();
  if (warp >= p.n_seqs * p.H) return;
  const int seq = warp / p.H, head = warp - seq * p.H;
  const HeadDesc d = p.desc[head];
  int ring_slot = p.j % d.z;
  if (p.acc != nullptr && d.w) {
    // Algorithm 2: the ring of a semantic head is a row buffer filled from slot 0.  First bring the
    // scores up to date with the attention of the layer's last decode (Algorithm 2, score
    // accumulation), then start the new token's score at zero.
    float* acc = p.acc + (size_t)warp * p.mr;
    if (p.pending) {
      const float* lg = p.logits + (size_t)warp * p.mr;
      const float2 ml = p.ml[warp];
      const float inv = 1.f / ml.y;
      const int n = p.static_valid + p.sem_slot;
      for (int i = lane; i < n; i += 32) {
        const int c = i < p.static_valid ? i : d.y + (i - p.static_valid);
        acc[c] += ex2(lg[c] - ml.x) * inv;
      }
    }
    ring_slot = p.sem_slot;
    if (lane == 0) acc[d.y + ring_slot] = 0.f;
  }
  uint4* dst = p.slab + ((size_t)seq * p.seq_slots + d.x + p.L + d.y + ring_slot) * kSlotU4;
  const uint4* src = (lane < 16 ? p.k_new : p.v_new) + (size_t)warp * 16 + (lane & 15);
  dst[lane] = *src;
}

}  // namespace

int decode_chunk_slots() { return kChunk; }

int decode_max_workers() {
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) {
    int v = 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0) sms = v;
  } else {
    cudaGetLastError();
  }
  if (sms < 148) sms = 148;  // size scratch for at least a full B200
  return sms * kWarps;
}

cudaError_t launch_decode(const DecodeParams& p_in, cudaStream_t st) {
  // Per-device set-up, done once; two host threads that meet here both do it (the calls are idempotent)
  // and publish the same value: 0 = not yet set up, else the device's worker count.
  static std::atomic<int> max_workers[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const bool cached = dev >= 0 && dev < 64;
  int workers = cached ? max_workers[dev].load(std::memory_order_acquire) : 0;
  if (workers == 0) {
    e = cudaFuncSetAttribute(ssd_decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    workers = decode_max_workers();
    if (cached) max_workers[dev].store(workers, std::memory_order_release);
  }
  DecodeParams p = p_in;
  const long total = (long)p.view.cum[p.view.H] * p.view.n_seqs;
  if (total < 1 || total > 0x7fffffffL) return cudaErrorInvalidValue;
  const long w = plan_workers(total, workers);
  p.split = make_split(total, w);
  const int grid = (int)((w + kWarps - 1) / kWarps);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  e = cudaLaunchKernelEx(&cfg, ssd_decode_kernel, p);
  count_launch();
  return e;
}

// Longest score row (M + R) whose logits a warp of the one-launch kernel can keep in shared memory.
int decode_layers_max_mr() { return ((227 * 1024 - kLayersSmemBytes) / (kWarps * 4)) & ~3; }

cudaError_t launch_fold_pending(float* acc, const float* logits, const float2* ml, const HeadDesc* desc, int n_seqs,
                                int H, int mr, int static_valid, int buffered, cudaStream_t st) {
  const int pairs = n_seqs * H;
  ssd_fold_pending_kernel<<<(pairs * 32 + 255) / 256, 256, 0, st>>>(acc, logits, ml, desc, pairs, H, mr, static_valid,
                                                                    buffered);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_decode_layers(const DecodeLayersParams& p, cudaStream_t st) {
  static std::atomic<int> n_sm[64] = {};   // 0 = this device is not set up yet (see launch_decode)
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const bool cached = dev >= 0 && dev < 64;
  int sms = cached ? n_sm[dev].load(std::memory_order_acquire) : 0;
  if (sms == 0) {
    e = cudaFuncSetAttribute(ssd_decode_layers_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             kLayersSmemBytes + kWarps * decode_layers_max_mr() * 4);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(ssd_decode_layers_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               kLayersSmemBytes + kWarps * decode_layers_max_mr() * 4);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    if (cached) n_sm[dev].store(sms, std::memory_order_release);
  }
  const long units = (long)p.n_layers * p.n_seqs * p.H;
  if (units < 1 || units > 0x3fffffffL || p.n_layers > kMaxLayersPerLaunch) return cudaErrorInvalidValue;
  if (p.mr < 0 || p.mr * (p.evict ? 3 : 1) > decode_layers_max_mr()) return cudaErrorInvalidValue;
  const long want = (units + kWarps - 1) / kWarps;            // no more CTAs than there are units for
  const int grid = (int)(want < sms ? want : sms);
  const int smem = kLayersSmemBytes + kWarps * ((p.mr + 3) & ~3) * 4 * (p.evict ? 3 : 1);
  if (p.evict) ssd_decode_layers_kernel<true><<<grid, kWarps * 32, smem, st>>>(p);
  else ssd_decode_layers_kernel<false><<<grid, kWarps * 32, smem, st>>>(p);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_append(const AppendParams& p, cudaStream_t st) {
  int warps = p.n_seqs * p.H;
  int grid = (warps * 32 + 255) / 256;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(256);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, ssd_append_kernel, p);
  count_launch();
  return e;
}

}  // namespace ssd
