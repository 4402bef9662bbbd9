// The decode-attention launch of ONE layer, written once for every slot format.
//
// Decode (consumer of Algorithm 1's output): for every (sequence, head) of one layer,
//   out = sum_i softmax_i(scale * <q, K_i>) V_i   over the slots that hold a token.
// It is a GEMV per head (1 flop per byte), so the kernel is built around keeping HBM busy and
// the instruction count per byte low, not around tensor cores:
//   * one CTA per SM, every streaming warp an independent worker.  The valid slots of the whole
//     layer form one logical stream of slots that is cut into equal shares, one per worker,
//     regardless of head type or length, so every SM moves the same bytes;
//   * a worker owns a ring of shared-memory stages.  Lane 0 fills them with bulk asynchronous
//     copies (cp.async.bulk, completion counted on an mbarrier per stage), one chunk of up to
//     kChunk slots per stage, and runs kStages chunks ahead of the arithmetic across head
//     boundaries; the query row of a head travels with the head's first chunk.  A stage is
//     pulled into registers and handed back to the copy engine before the arithmetic starts;
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
// Fused append: the newest token's K/V rows are taken from the caller's k_new / v_new instead of
// the slab, and the worker that consumes the chunk holding the token's ring slot writes the slot
// into the slab for later steps.  Nothing reads that slab slot during the launch, so no ordering
// is needed, and the per-layer append launch disappears.
// Every wait on an mbarrier is bounded: a warp that gives up raises a bit in the status word,
// waits (bounded again) for its other copies in flight and leaves.
//
// What depends on how a slot stores its two rows is a policy class F:
//   kWarps, kStages, kChunk     streaming warps per CTA, stages per warp, slots per stage
//   kSlot                       bytes per slot
//   kNewBytes                   stage bytes set aside for the newest token's rows as the caller passes
//                               them (0: they are copied straight into the token's slot of the stage,
//                               and the slab is copied around that slot)
//   Rows, load_q, load_stage, fold_stage     a stage's slots in registers, and the arithmetic on them
//   store_new                   put the newest token's slot into the slab (and, with kNewBytes > 0,
//                               into its place in the stage, converted)
//   post_acc, write_out         a lane's 16 output dimensions into a mailbox / the output row
#pragma once

#include <atomic>

#include "ssd_internal.cuh"
#include "ssd_device.cuh"

namespace ssd {

constexpr int kQBytes = kHeadDim * 2;    // a bf16 row of q, k_new, v_new, out

// Shared-memory geometry of a CTA: [rings | stage barriers, finisher's two | mailboxes | arrival counters]
template <class F>
struct Geo {
  static constexpr int kThreads = (F::kWarps + 1) * 32;               // plus one finisher warp
  static constexpr int kStageQ = F::kChunk * F::kSlot;                // where the query row sits in a stage
  static constexpr int kStageNew = kStageQ + kQBytes;                 // and (kNewBytes > 0) the newest token's rows
  static constexpr int kStageBytes = kStageNew + F::kNewBytes;
  static constexpr int kRingBytes = F::kWarps * F::kStages * kStageBytes;
  static constexpr int kBarBytes = (F::kWarps * F::kStages + 2) * 8;
  static constexpr int kMailBoxes = F::kWarps * 2 + 2;                // two partials per worker, two for the CTA
  static constexpr int kMailBytes = kMailBoxes * kPartialFloats * 4;
  static constexpr int kCountBytes = F::kWarps * 2 * 4;               // arrival counter per (first worker, slot)
  static constexpr int kSmemBytes = kRingBytes + kBarBytes + kMailBytes + kCountBytes;
  static_assert(kSmemBytes <= 227 * 1024, "stage rings exceed the shared memory of an SM");
  static_assert(kStageBytes % 16 == 0 && F::kSlot % 16 == 0, "bulk copies move multiples of 16 bytes");
  static_assert(kBarBytes % 16 == 0, "mailboxes are read as float4");
};

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

__device__ __forceinline__ uint32_t pack_bf16(float2 a, float inv) {
  __nv_bfloat162 t = __floats2bfloat162_rn(a.x * inv, a.y * inv);
  return *reinterpret_cast<uint32_t*>(&t);
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

// Where the logits of a chunk go when the scores of semantic heads are being accumulated
// (Algorithm 2): row = the head's logit row (null: nothing to record), slot s of the chunk is valid
// slot i0 + s of the head; valid slots below `skip` are prompt slots (not scored) and those from
// `ring_from` on sit `ring_shift` entries further (unused static capacity in between).
struct LogitSink {
  float* row;
  int i0, skip, ring_from, ring_shift;
};

// Algorithm 2, score accumulation, deferred by one step: the weights of the layer's previous decode go into
// the scores at the start of the layer's next launch (nothing in that launch reads the scores), and the
// token being appended starts at zero.  Run by the finisher warp of every thread block, which share the
// pairs; entry c of a score row is static slot c or, from the static capacity on, buffer slot c - capacity.
__device__ inline void fold_scores(const DecodeParams& p, int lane) {
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
template <class F>
__device__ void finisher(const DecodeParams& p, const unsigned char* smem, int lane) {
  using G = Geo<F>;
  constexpr int kWarps = F::kWarps, kStages = F::kStages, kRingBytes = G::kRingBytes, kBarBytes = G::kBarBytes;
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

template <class F>
__global__ void __launch_bounds__(Geo<F>::kThreads, 1) ssd_decode_kernel(const __grid_constant__ DecodeParams p) {
  using G = Geo<F>;
  constexpr int kWarps = F::kWarps, kStages = F::kStages, kChunk = F::kChunk, kSlot = F::kSlot;
  constexpr int kStageBytes = G::kStageBytes, kRingBytes = G::kRingBytes, kBarBytes = G::kBarBytes;
  constexpr int kMailBytes = G::kMailBytes, kStageQ = G::kStageQ, kStageNew = G::kStageNew;
  constexpr bool kNewInPlace = F::kNewBytes == 0;
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
    finisher<F>(p, smem, lane);
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
    pl.hbase = reinterpret_cast<const unsigned char*>(p.slab) + ((size_t)w.seq * v.seq_slots + v.head[w.head].x) * kSlot;
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
      mbar_expect_tx(bar, (uint32_t)(n * kSlot + (pl.begin ? kQBytes : 0) + ((has_fresh && !kNewInPlace) ? 2 * kQBytes : 0)));
      // valid slots [a, a + len) of the head into the stage from slot `at` on
      auto copy_range = [&](int a, int len, int at) {
        if (len <= 0) return;
        if (v.contig) {
          bulk_g2s(dst + (uint32_t)at * kSlot, pl.hbase + (size_t)a * kSlot, (uint32_t)len * kSlot, bar);
        } else {
          chunk_runs(v, pl.head, a, len, [&](int src, int d, int l) {
            bulk_g2s(dst + (uint32_t)(at + d) * kSlot, pl.hbase + (size_t)src * kSlot, (uint32_t)l * kSlot, bar);
          });
        }
      };
      if (has_fresh && kNewInPlace) {    // the slab is copied around the newest token's slot
        copy_range(pl.i, fresh - pl.i, 0);
        copy_range(fresh + 1, pl.i + n - fresh - 1, fresh + 1 - pl.i);
      } else {
        copy_range(pl.i, n, 0);
      }
    }
    if (what & 2) {
      if (has_fresh) {
        // the newest token's rows: into its slot of the stage, or (a format that converts them) behind the query row
        const uint32_t at = kNewInPlace ? (uint32_t)(fresh - pl.i) * kSlot : (uint32_t)kStageNew;
        bulk_g2s(dst + at, p.k_new + pl.row, kQBytes, bar);
        bulk_g2s(dst + at + kQBytes, p.v_new + pl.row, kQBytes, bar);
      }
      if (pl.begin) bulk_g2s(dst + kStageQ, reinterpret_cast<const unsigned char*>(p.q) + pl.row, kQBytes, bar);
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
    unsigned char* sb = ring + (size_t)stage * kStageBytes;
    if (begin) {
      F::load_q(sb + kStageQ, l8, p.scale_log2, q);
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
    typename F::Rows rows;
    if (kNewInPlace) F::load_stage(sb, n, grp, l8, rows);
    if (p.new_j >= 0) {
      // fused append: the chunk that carries the newest token also stores it in the slab
      const int s_new = fresh - cons.i;
      if (s_new >= 0 && s_new < n) {
        unsigned char* in_slab = reinterpret_cast<unsigned char*>(const_cast<uint4*>(p.slab)) +
                                 ((size_t)cons.seq * v.seq_slots + v.head[cons.head].x + fresh_phys) * kSlot;
        F::store_new(sb + s_new * kSlot, sb + kStageNew, in_slab, lane);
      }
    }
    if (!kNewInPlace) F::load_stage(sb, n, grp, l8, rows);   // after the newest token's slot has been written
    __syncwarp();          // every lane has its rows in registers: the stage may be refilled
    --ahead;
    if (more) {
      fire_chunk(next, stage, 3);
      advance(prod, next.n);
      ++ahead;
    }
    F::fold_stage(rows, n, grp, l8, q, st, sink);

    const int i1 = cons.i + n;
    if (i1 == cons.vh || cons.g + n == cons.g_end) {
      // end of this worker's piece of the head: merge the four groups (lanes l, l^8, l^16, l^24
      // hold the same 16 output dims), then write the output, or post a partial to the finisher
      State tot = st;
      state_merge_lane(tot, 8);
      state_merge_lane(tot, 16);
      if (piece_i0 == 0 && i1 == cons.vh) {
        if (grp == 0) F::write_out(p.out + ((size_t)cons.seq * v.H + cons.head) * kHeadDim, tot, l8);
        if (p.ml != nullptr && lane == 0) p.ml[(size_t)cons.seq * v.H + cons.head] = make_float2(tot.m, tot.l);
      } else {
        // post the partial; the worker that posts a head's last piece in this CTA merges them
        float* P = mail + (size_t)(2 * warp + (leading ? 0 : 1)) * kPartialFloats;
        if (lane == 0) {
          P[0] = tot.m;
          P[1] = tot.l;
        }
        if (grp == 0) F::post_acc(P + 4, tot, l8);
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
// Workers (streaming warps) a launch of this format may use on the current device.
template <class F>
int decode_workers_on_device() {
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) {
    int v = 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0) sms = v;
  } else {
    cudaGetLastError();
  }
  if (sms < 148) sms = 148;  // size scratch for at least a full B200
  return sms * F::kWarps;
}

template <class F>
cudaError_t launch_decode_format(const DecodeParams& p_in, cudaStream_t st) {
  // Per-device set-up, done once; two host threads that meet here both do it (the calls are idempotent)
  // and publish the same value: 0 = not yet set up, else the device's worker count.
  static std::atomic<int> max_workers[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const bool cached = dev >= 0 && dev < 64;
  int workers = cached ? max_workers[dev].load(std::memory_order_acquire) : 0;
  if (workers == 0) {
    e = cudaFuncSetAttribute(ssd_decode_kernel<F>, cudaFuncAttributeMaxDynamicSharedMemorySize, Geo<F>::kSmemBytes);
    if (e != cudaSuccess) return e;
    workers = decode_workers_on_device<F>();
    if (cached) max_workers[dev].store(workers, std::memory_order_release);
  }
  DecodeParams p = p_in;
  const long total = (long)p.view.cum[p.view.H] * p.view.n_seqs;
  if (total < 1 || total > 0x7fffffffL) return cudaErrorInvalidValue;
  const long w = plan_workers(total, workers);
  p.split = make_split(total, w);
  const int grid = (int)((w + F::kWarps - 1) / F::kWarps);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(Geo<F>::kThreads);
  cfg.dynamicSmemBytes = Geo<F>::kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  e = cudaLaunchKernelEx(&cfg, ssd_decode_kernel<F>, p);
  count_launch();
  return e;
}

}  // namespace ssd
