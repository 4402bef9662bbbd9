// Decode attention over the head-decoupled compressed KV store in its bf16 format (512-byte slots,
// [K row | V row]), and the per-step append/evict.
//   ssd_decode_kernel<Bf16Slots>   one layer per launch: the kernel of ssd_decode_layer.cuh with the
//                                  arithmetic of this format;
//   ssd_decode_layers_kernel       a whole step (every layer) in one launch;
//   ssd_fold_pending_kernel, ssd_append_kernel   the small kernels of the two-launch forms.
// Arithmetic per chunk of slots: the warp works as four groups of 8 lanes, group g taking slots g,
// g + 4, ...; a lane covers 16 of the 128 dimensions with two 128-bit reads per row, packed
// two-wide fp32 FMAs, three shuffles per dot product, and an online softmax in fp32 (base-2
// exponent, scale folded into q).
#include <atomic>

#include "ssd_decode_layer.cuh"


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
constexpr int kStages = SSD_DECODE_STAGES;
constexpr int kChunk = SSD_DECODE_CHUNK;             // slots per stage
constexpr int kGroups = 4;                           // 8-lane groups of a warp
constexpr int kPer = kChunk / kGroups;               // slots of a stage each group takes
constexpr int kU = kPer % 4 == 0 ? 4 : (kPer % 3 == 0 ? 3 : (kPer % 2 == 0 ? 2 : 1));   // slots a group folds in at a time
constexpr int kStageBytes = kChunk * kSlotBytes + kQBytes;
constexpr int kRingBytes = kWarps * kStages * kStageBytes;

static_assert(kChunk % kGroups == 0 && kPer % kU == 0, "a stage is folded in groups of kGroups * kU slots");
static_assert((kWarps * kStages) % 2 == 0, "keeps the mailboxes 16-byte aligned");

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

// lanes 0..7 write the row: 16 bytes at dimension 8*l8 and 16 bytes at dimension 64 + 8*l8
__device__ __forceinline__ void write_out(__nv_bfloat16* out, const State& st, int l8) {
  const float inv = 1.f / st.l;
  uint4* o = reinterpret_cast<uint4*>(out);
  o[l8] = make_uint4(pack_bf16(st.acc[0], inv), pack_bf16(st.acc[1], inv), pack_bf16(st.acc[2], inv),
                     pack_bf16(st.acc[3], inv));
  o[8 + l8] = make_uint4(pack_bf16(st.acc[4], inv), pack_bf16(st.acc[5], inv), pack_bf16(st.acc[6], inv),
                         pack_bf16(st.acc[7], inv));
}

// The 512-byte slot format as the one-layer kernel sees it.
struct Bf16Slots {
  static constexpr int kWarps = ssd::kWarps, kStages = ssd::kStages, kChunk = ssd::kChunk;
  static constexpr int kSlot = kSlotBytes;
  static constexpr int kNewBytes = 0;      // the newest token's rows are copied straight into its slot of the stage
  using Rows = ssd::Rows;
  // the lane's 16 dimensions of the query row, widened and scaled
  static __device__ __forceinline__ void load_q(const unsigned char* qrow, int l8, float scale_log2, float2 (&q)[8]) {
    const uint4 qa = reinterpret_cast<const uint4*>(qrow)[l8], qb = reinterpret_cast<const uint4*>(qrow)[8 + l8];
    const float2 sc = make_float2(scale_log2, scale_log2);
    q[0] = __fmul2_rn(widen2(qa.x), sc); q[1] = __fmul2_rn(widen2(qa.y), sc);
    q[2] = __fmul2_rn(widen2(qa.z), sc); q[3] = __fmul2_rn(widen2(qa.w), sc);
    q[4] = __fmul2_rn(widen2(qb.x), sc); q[5] = __fmul2_rn(widen2(qb.y), sc);
    q[6] = __fmul2_rn(widen2(qb.z), sc); q[7] = __fmul2_rn(widen2(qb.w), sc);
  }
  static __device__ __forceinline__ void load_stage(const unsigned char* sb, int n, int grp, int l8, Rows& r) {
    ssd::load_stage(reinterpret_cast<const uint4*>(sb), n, grp, l8, r);
  }
  static __device__ __forceinline__ void fold_stage(const Rows& r, int n, int grp, int l8, const float2 (&q)[8], State& st,
                                                    const LogitSink& sink) {
    ssd::fold_stage(r, n, grp, l8, q, st, sink);
  }
  // the slot already stands in the stage as it will in the slab
  static __device__ __forceinline__ void store_new(const unsigned char* in_stage, const unsigned char*, unsigned char* in_slab,
                                                   int lane) {
    reinterpret_cast<uint4*>(in_slab)[lane] = reinterpret_cast<const uint4*>(in_stage)[lane];
  }
  // lane l8 of a group holds dimensions [8 * l8, 8 * l8 + 8) and [64 + 8 * l8, 64 + 8 * l8 + 8)
  static __device__ __forceinline__ void post_acc(float* acc128, const State& tot, int l8) {
    float4* lo = reinterpret_cast<float4*>(acc128 + 8 * l8);
    float4* hi = reinterpret_cast<float4*>(acc128 + 64 + 8 * l8);
    lo[0] = make_float4(tot.acc[0].x, tot.acc[0].y, tot.acc[1].x, tot.acc[1].y);
    lo[1] = make_float4(tot.acc[2].x, tot.acc[2].y, tot.acc[3].x, tot.acc[3].y);
    hi[0] = make_float4(tot.acc[4].x, tot.acc[4].y, tot.acc[5].x, tot.acc[5].y);
    hi[1] = make_float4(tot.acc[6].x, tot.acc[6].y, tot.acc[7].x, tot.acc[7].y);
  }
  static __device__ __forceinline__ void write_out(__nv_bfloat16* out, const State& st, int l8) { ssd::write_out(out, st, l8); }
};

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

int decode_max_workers() { return decode_workers_on_device<Bf16Slots>(); }

cudaError_t launch_decode(const DecodeParams& p, cudaStream_t st) { return launch_decode_format<Bf16Slots>(p, st); }

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
