// Decode attention over the head-decoupled compressed KV store in its bf16 format (512-byte slots,
// [K row | V row]), and the per-step append/evict.
//   ssd_decode_kernel<Bf16Slots>   one layer per launch: the kernel of ssd_decode_layer.cuh with the
//                                  arithmetic of this format;
//   ssd_decode_layers_kernel<Bf16Slots, kEvict>   a whole step (every layer) in one launch: the kernel of
//                                  ssd_decode_step.cuh, likewise;
//   ssd_fold_pending_kernel, ssd_append_kernel   the small kernels of the two-launch forms.
// Arithmetic per chunk of slots: the warp works as four groups of 8 lanes, group g taking slots g,
// g + 4, ...; a lane covers 16 of the 128 dimensions with two 128-bit reads per row, packed
// two-wide fp32 FMAs, three shuffles per dot product, and an online softmax in fp32 (base-2
// exponent, scale folded into q).
#include <atomic>

#include "ssd_decode_step.cuh"


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
  static constexpr bool kScores = true;    // serves the row-buffer modes of the one-launch step
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
int decode_layers_max_mr() { return step_max_mr<Bf16Slots>(); }

cudaError_t launch_fold_pending(float* acc, const float* logits, const float2* ml, const HeadDesc* desc, int n_seqs,
                                int H, int mr, int static_valid, int buffered, cudaStream_t st) {
  const int pairs = n_seqs * H;
  ssd_fold_pending_kernel<<<(pairs * 32 + 255) / 256, 256, 0, st>>>(acc, logits, ml, desc, pairs, H, mr, static_valid,
                                                                    buffered);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_decode_layers(const DecodeLayersParams& p, cudaStream_t st) {
  return launch_decode_step_format<Bf16Slots>(p, st);
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
