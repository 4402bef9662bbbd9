// A whole decode step (every layer's fused append + attention) in ONE launch, written once for every slot
// format (the policy class F of ssd_decode_layer.cuh).
//
// With all layers in one launch there are tens of thousands of heads to go round, so no head needs to
// be cut: the unit of work is one whole head of one (layer, sequence), units are handed out in stream
// order from a global counter to whichever warp asks next (warps on slower SMs simply take fewer), and a
// head is finished in the registers of the warp that streamed it.  No partials, no mailboxes, no
// finisher, no barrier after start-up.  A warp's copy pipeline runs on across unit boundaries: the next
// unit is claimed while the current one streams, and its first chunks are in flight before the current
// head's arithmetic ends.  In the row-buffer modes (formats with F::kScores) the warp that streamed a
// semantic head also adds the step's attention weights to the head's scores (Algorithm 2) or, with a
// buffer of one token, re-selects on the spot (kEvict: Algorithm 1 taken literally).
#pragma once

#include "ssd_decode_layer.cuh"

namespace ssd {

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

template <class F>
__device__ __forceinline__ void unit_load(const DecodeLayersParams& p, int u, Unit& U) {
  const int pairs = p.n_seqs * p.H;
  const int layer = u / pairs, pair = u - layer * pairs;
  const int seq = pair / p.H, head = pair - seq * p.H;
  const LayerState& ls = p.layer[layer];
  const HeadDesc d = __ldg(ls.desc + head);
  U.u = u;
  U.scored = (F::kScores && p.acc != nullptr && d.w) ? 1 : 0;
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
            ((size_t)ls.first_slot + (size_t)seq * ls.seq_slots + d.x) * F::kSlot;
  U.row = ((size_t)layer * pairs + pair) * kQBytes;
}

// Shared memory of a CTA: [rings | stage barriers | a 4-entry FIFO of unit ids per warp | row-buffer mode: the warps' logit rows]
template <class F>
struct StepGeo {
  static constexpr int kRingBytes = F::kWarps * F::kStages * Geo<F>::kStageBytes;
  static constexpr int kSmemBytes = kRingBytes + F::kWarps * F::kStages * 8 + F::kWarps * 4 * 4;
  static_assert(kSmemBytes <= 227 * 1024, "stage rings exceed the shared memory of an SM");
};

// kEvict: Algorithm 1 taken literally (a row buffer of one token, re-selected in the same launch).
template <class F, bool kEvict>
__global__ void __launch_bounds__(F::kWarps * 32, 1) ssd_decode_layers_kernel(const __grid_constant__ DecodeLayersParams p) {
  constexpr int kWarps = F::kWarps, kStages = F::kStages, kChunk = F::kChunk, kSlot = F::kSlot, kSlotU4 = F::kSlot / 16;
  constexpr int kStageBytes = Geo<F>::kStageBytes, kStageQ = Geo<F>::kStageQ, kStageNew = Geo<F>::kStageNew;
  constexpr int kRingBytes = StepGeo<F>::kRingBytes, kLayersSmemBytes = StepGeo<F>::kSmemBytes;
  constexpr bool kNewInPlace = F::kNewBytes == 0;
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
  unit_load<F>(p, u, PU);
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
      mbar_expect_tx(bar, (uint32_t)(n * kSlot + (begin ? kQBytes : 0) + ((has_fresh && !kNewInPlace) ? 2 * kQBytes : 0)));
      // valid slots [a, a + len) of the head into the stage from slot `at` on
      auto copy_range = [&](int a, int len, int at) {
        if (len <= 0) return;
        if (PU.contig) {
          bulk_g2s(dst + (uint32_t)at * kSlot, PU.hbase + (size_t)a * kSlot, (uint32_t)len * kSlot, bar);
          return;
        }
        const int l0[3] = {0, PU.pv, PU.pv + PU.sv};          // logical start of each run
        const int l1[3] = {PU.pv, PU.pv + PU.sv, PU.vh};      // and end
        const int p0[3] = {0, p.L, p.L + PU.y};               // physical start
#pragma unroll
        for (int r = 0; r < 3; ++r) {
          const int lo = a > l0[r] ? a : l0[r], hi = a + len < l1[r] ? a + len : l1[r];
          if (hi > lo)
            bulk_g2s(dst + (uint32_t)(at + lo - a) * kSlot, PU.hbase + (size_t)(p0[r] + lo - l0[r]) * kSlot,
                     (uint32_t)(hi - lo) * kSlot, bar);
        }
      };
      if (has_fresh && kNewInPlace) {    // the slab is copied around the newest token's slot
        copy_range(pi, PU.fresh - pi, 0);
        copy_range(PU.fresh + 1, pi + n - PU.fresh - 1, PU.fresh + 1 - pi);
      } else {
        copy_range(pi, n, 0);
      }
      if (has_fresh) {
        // the newest token's rows: into its slot of the stage, or (a format that converts them) behind the query row
        const uint32_t at = kNewInPlace ? (uint32_t)(PU.fresh - pi) * kSlot : (uint32_t)kStageNew;
        bulk_g2s(dst + at, p.k_new + PU.row, kQBytes, bar);
        bulk_g2s(dst + at + kQBytes, p.v_new + PU.row, kQBytes, bar);
      }
      if (begin) bulk_g2s(dst + kStageQ, p.q + PU.row, kQBytes, bar);
    }
    pi += n;
    ++ahead;
    if (pi == PU.vh) {                   // on to the unit asked for earlier, and ask for the one after
      const int nu = __shfl_sync(FULL, raw_next, 0);
      if (nu < n_units) {
        ask();
        unit_load<F>(p, nu, PU);
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
      unit_load<F>(p, fifo[consumed & 3], CU);
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
    unsigned char* sb = ring + (size_t)stage * kStageBytes;
    if (begin) {
      F::load_q(sb + kStageQ, l8, p.scale_log2, q);
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
    typename F::Rows rows;
    if (kNewInPlace) F::load_stage(sb, n, grp, l8, rows);
    {
      // the chunk that carries the newest token also stores it in the slab
      const int s_new = CU.fresh - ci;
      if (s_new >= 0 && s_new < n)
        F::store_new(sb + s_new * kSlot, sb + kStageNew, const_cast<unsigned char*>(CU.hbase) + (size_t)CU.phys * kSlot, lane);
    }
    if (!kNewInPlace) F::load_stage(sb, n, grp, l8, rows);   // after the newest token's slot has been written
    __syncwarp();          // every lane has its rows in registers: the stage may be refilled
    --ahead;
    if (feeding) issue(stage);
    F::fold_stage(rows, n, grp, l8, q, st, sink);
    ci += n;
    if (ci == CU.vh) {
      // the head is complete: merge the four groups and write the output row
      State tot = st;
      state_merge_lane(tot, 8);
      state_merge_lane(tot, 16);
      if (grp == 0) F::write_out(reinterpret_cast<__nv_bfloat16*>(reinterpret_cast<unsigned char*>(p.out) + CU.row), tot, l8);
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
// Longest score row (M + R) whose logits a warp of the one-launch kernel can keep in shared memory.
template <class F>
constexpr int step_max_mr() { return ((227 * 1024 - StepGeo<F>::kSmemBytes) / (F::kWarps * 4)) & ~3; }

// F::kScores: the format serves the row-buffer modes (score rows in shared memory, the kEvict instance)
template <class F>
cudaError_t launch_decode_step_format(const DecodeLayersParams& p, cudaStream_t st) {
  constexpr bool kScores = F::kScores;
  static std::atomic<int> n_sm[64] = {};   // 0 = this device is not set up yet (see launch_decode_format)
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const bool cached = dev >= 0 && dev < 64;
  int sms = cached ? n_sm[dev].load(std::memory_order_acquire) : 0;
  constexpr int kBase = StepGeo<F>::kSmemBytes;
  constexpr int kMaxMr = kScores ? step_max_mr<F>() : 0;
  if (sms == 0) {
    e = cudaFuncSetAttribute(ssd_decode_layers_kernel<F, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             kBase + F::kWarps * kMaxMr * 4);
    if (kScores && e == cudaSuccess)
      e = cudaFuncSetAttribute(ssd_decode_layers_kernel<F, kScores>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               kBase + F::kWarps * kMaxMr * 4);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    if (cached) n_sm[dev].store(sms, std::memory_order_release);
  }
  const long units = (long)p.n_layers * p.n_seqs * p.H;
  if (units < 1 || units > 0x3fffffffL || p.n_layers > kMaxLayersPerLaunch) return cudaErrorInvalidValue;
  if (!kScores && (p.acc != nullptr || p.evict)) return cudaErrorInvalidValue;
  if (p.mr < 0 || p.mr * (p.evict ? 3 : 1) > kMaxMr) return cudaErrorInvalidValue;
  const long want = (units + F::kWarps - 1) / F::kWarps;      // no more CTAs than there are units for
  const int grid = (int)(want < sms ? want : sms);
  const int smem = kBase + F::kWarps * ((p.mr + 3) & ~3) * 4 * (p.evict ? 3 : 1);
  if (kScores && p.evict) ssd_decode_layers_kernel<F, kScores><<<grid, F::kWarps * 32, smem, st>>>(p);
  else ssd_decode_layers_kernel<F, false><<<grid, F::kWarps * 32, smem, st>>>(p);
  count_launch();
  return cudaGetLastError();
}

}  // namespace ssd
