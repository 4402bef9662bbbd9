// 8-bit K/V: an extension the paper only cites as related work (Sec. 2, "KV Cache Compression").  The same
// head-decoupled store, with every cached row held as 128 E4M3 codes (OCP 8-bit floating point: 4 exponent
// bits, bias 7, 3 mantissa bits, largest magnitude 448) and one float32 scale per row,
//   scale = max|x| / 448,   code = E4M3(x / scale)   (round to nearest even, saturating; float32 arithmetic),
// so a slot is [K codes 128 B | V codes 128 B | K scale | V scale | 8 B unused] = 272 bytes instead of 512.
// A row is quantised once, when it enters the cache (by the gather of ssd_compress, or by the decode launch
// that appends it), so what later steps read does not depend on when they read it.
//   ssd_quantize_rows_kernel   the quantiser on its own (parity of the codes, bit for bit)
//   ssd_gather_q8_kernel       ssd_compress's gather, quantising on the way into the slab
//   ssd_decode_layers_kernel<Q8Slots<12, 24>>   fused append + decode attention of every layer in one launch: the
//                              kernel of ssd_decode_step.cuh (whole heads handed out to warps from a counter) with
//                              the arithmetic of this format: codes are widened with cvt.rn.f16x2.e4m3x2 (exact), all
//                              arithmetic in float32, the row scales applied to the logit and to the softmax weight
//   ssd_decode_kernel<Q8Slots<..>>   one layer per launch: the equal-shares kernel of ssd_decode_layer.cuh with the
//                              same arithmetic (decode alone, or fused with the append)
#include <cuda_fp16.h>

#include <atomic>

#include "ssd_decode_step.cuh"

namespace ssd {

namespace {

constexpr int kQ8SlotBytes = 272;

// two floats -> two E4M3 codes (a in the low byte)
__device__ __forceinline__ uint32_t e4m3x2(float a, float b) {
  uint16_t r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(b), "f"(a));
  return r;
}

// 8 bf16 values of a row (one uint4) -> 8 codes (uint2), given the row's scale
__device__ __forceinline__ uint2 quantize8(const uint4& raw, float scale) {
  const float s = scale > 0.f ? scale : 1.f;
  const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
  uint32_t c[4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
    c[i] = e4m3x2(__fdiv_rn(__uint_as_float(w[i] << 16), s), __fdiv_rn(__uint_as_float(w[i] & 0xffff0000u), s));
  return make_uint2(c[0] | (c[1] << 16), c[2] | (c[3] << 16));
}

__device__ __forceinline__ float amax8(const uint4& raw) {
  const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
  float m = 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i)
    m = fmaxf(m, fmaxf(fabsf(__uint_as_float(w[i] << 16)), fabsf(__uint_as_float(w[i] & 0xffff0000u))));
  return m;
}

// A row is held by 16 consecutive lanes (8 values each): its scale, the same in all 16 lanes.
__device__ __forceinline__ float row_scale16(const uint4& raw) {
  float m = amax8(raw);
#pragma unroll
  for (int o = 8; o >= 1; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  return __fdiv_rn(m, 448.f);
}

// ----------------------------------------------------------------------------- the quantiser on its own
__global__ void __launch_bounds__(256) ssd_quantize_rows_kernel(const uint4* __restrict__ rows, long long n_rows,
                                                                uint2* __restrict__ codes, float* __restrict__ scales) {
  const long long hw = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 4;   // one half-warp per row
  const int l16 = threadIdx.x & 15;
  const bool ok = hw < n_rows;
  const uint4 raw = ok ? rows[hw * 16 + l16] : make_uint4(0, 0, 0, 0);
  const float scale = row_scale16(raw);
  if (!ok) return;
  codes[hw * 16 + l16] = quantize8(raw, scale);
  if (l16 == 0) scales[hw] = scale;
}

// ----------------------------------------------------------------------------- gather into 272-byte slots
// One warp per destination slot, two slots at a time: lanes 0-15 quantise the K row, lanes 16-31 the V row.
// The work is shared out as in ssd_gather_kernel: the thread blocks of the last y copy the static slots of
// semantic heads once the selection kernel has completed, all others what does not depend on the selection.
__global__ void __launch_bounds__(256) ssd_gather_q8_kernel(const GatherParams p) {
  const int pair = blockIdx.x;
  const int seq = pair / p.H, head = pair - seq * p.H;
  const HeadDesc d = p.desc[head];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int ctx = p.L + p.n0;
  unsigned char* dst0 = reinterpret_cast<unsigned char*>(p.slab) + ((size_t)seq * p.seq_slots + d.x) * kQ8SlotBytes;
  const uint4* src = (lane < 16 ? p.k_full : p.v_full) + (size_t)pair * ctx * 16 + (lane & 15);
  auto put = [&](int s, const uint4& raw) {        // the whole warp together (the row scale is a warp reduction)
    const float scale = row_scale16(raw);
    unsigned char* dst = dst0 + (size_t)s * kQ8SlotBytes;
    reinterpret_cast<uint2*>(dst)[lane] = quantize8(raw, scale);           // K codes at 0, V codes at 128
    if ((lane & 15) == 0) reinterpret_cast<float*>(dst + 256)[lane >> 4] = scale;
  };
  const bool selected = blockIdx.y == gridDim.y - 1;
  int s, end, stride;
  if (selected) {
    const bool work = d.w && p.static_valid > 0;
    if (!work && pair != 0) return;
    pdl_wait_predecessor();                        // (pair 0 waits in any case: the launch must not complete before
    if (!work) return;                             // the selection has)
    s = p.L + warp; end = p.L + p.static_valid; stride = 8;
  } else {
    s = blockIdx.y * 8 + warp; end = p.L + d.y + d.z; stride = (gridDim.y - 1) * 8;
  }
  for (; s < end; s += 2 * stride) {
    const int s2 = s + stride;
    const bool a = gather_slot_selected(p, d, s) == selected;
    const bool b = s2 < end && gather_slot_selected(p, d, s2) == selected;
    const int pa = a ? gather_source_row(p, d, pair, s) : -1;               // the same for the whole warp
    const int pb = b ? gather_source_row(p, d, pair, s2) : -1;
    uint4 ra = make_uint4(0, 0, 0, 0), rb = ra;
    if (pa >= 0) ra = src[(size_t)pa * 16];
    if (pb >= 0) rb = src[(size_t)pb * 16];
    if (pa >= 0) put(s, ra);
    if (pb >= 0) put(s2, rb);
  }
}

// ----------------------------------------------------------------------------- decode over 272-byte slots
#ifndef SSD_Q8_WARPS
#define SSD_Q8_WARPS 12           // the one-launch step: streaming warps per CTA ...
#endif
#ifndef SSD_Q8_CHUNK
#define SSD_Q8_CHUNK 24           // ... and slots per stage (6528 bytes per copy in steady state); 2 stages
#endif
constexpr int kGroups = 4;                 // 8-lane groups of a warp; group g takes slots g, g + 4, ..

// slots a group folds in at a time, of the kPer it takes from a stage
template <int kPer>
struct FoldWidth {
  static constexpr int value = kPer % 4 == 0 ? 4 : (kPer % 3 == 0 ? 3 : (kPer % 2 == 0 ? 2 : 1));
};
constexpr int kRowBytes = kHeadDim * 2;    // a bf16 row of q, k_new, v_new, out


// 4 codes (one 32-bit word) -> 4 floats, exactly
__device__ __forceinline__ void widen4(uint32_t w, float2& lo, float2& hi) {
  uint32_t a, b;
  asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(a) : "h"((uint16_t)(w & 0xffffu)));
  asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(b) : "h"((uint16_t)(w >> 16)));
  lo = __half22float2(*reinterpret_cast<const __half2*>(&a));
  hi = __half22float2(*reinterpret_cast<const __half2*>(&b));
}

// The rows of a stage as one lane holds them: slot 4*u + grp, 16 codes of K and of V (dimensions
// [16*l8, 16*l8 + 16)) and the two row scales.
template <int kPer>
struct Q8Rows {
  uint4 k[kPer], v[kPer];
  float ks[kPer], vs[kPer];
};

template <int kPer>
__device__ __forceinline__ void q8_load_stage(const unsigned char* __restrict__ sb, int n, int grp, int l8, Q8Rows<kPer>& r) {
#pragma unroll
  for (int u = 0; u < kPer; ++u) {
    const int slot = kGroups * u + grp;
    const unsigned char* s = sb + slot * kQ8SlotBytes;
    if (slot < n) {
      r.k[u] = reinterpret_cast<const uint4*>(s)[l8];
      r.v[u] = reinterpret_cast<const uint4*>(s + 128)[l8];
      const float2 sc = *reinterpret_cast<const float2*>(s + 256);
      r.ks[u] = sc.x;
      r.vs[u] = sc.y;
    } else {
      r.k[u] = r.v[u] = make_uint4(0, 0, 0, 0);
      r.ks[u] = r.vs[u] = 0.f;
    }
  }
}

__device__ __forceinline__ float q8_dot16(const uint4& k, const float2 (&q)[8]) {
  const uint32_t w[4] = {k.x, k.y, k.z, k.w};
  float2 a = make_float2(0.f, 0.f), b = make_float2(0.f, 0.f);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float2 lo, hi;
    widen4(w[i], lo, hi);
    a = __ffma2_rn(lo, q[2 * i], a);
    b = __ffma2_rn(hi, q[2 * i + 1], b);
  }
  return (a.x + a.y) + (b.x + b.y);
}

__device__ __forceinline__ void q8_axpy16(float p, const uint4& v, float2 (&acc)[8]) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
  const float2 pp = make_float2(p, p);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float2 lo, hi;
    widen4(w[i], lo, hi);
    acc[2 * i] = __ffma2_rn(pp, lo, acc[2 * i]);
    acc[2 * i + 1] = __ffma2_rn(pp, hi, acc[2 * i + 1]);
  }
}

template <int kPer>
__device__ __forceinline__ void q8_fold_stage(const Q8Rows<kPer>& r, int n, int grp, const float2 (&q)[8], State& st) {
  constexpr int kU = FoldWidth<kPer>::value;
#pragma unroll
  for (int s = 0; s < kPer; s += kU) {
    if (kGroups * s >= n) break;
    float x[kU];
#pragma unroll
    for (int u = 0; u < kU; ++u) x[u] = q8_dot16(r.k[s + u], q);
#pragma unroll
    for (int off = 4; off >= 1; off >>= 1) {
#pragma unroll
      for (int u = 0; u < kU; ++u) x[u] += __shfl_xor_sync(0xffffffffu, x[u], off);
    }
    float mn = st.m;
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      x[u] = kGroups * (s + u) + grp < n ? x[u] * r.ks[s + u] : kNegBig;     // the K row's scale
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
    for (int u = 0; u < kU; ++u) q8_axpy16(p[u] * r.vs[s + u], r.v[s + u], st.acc);   // the V row's scale
  }
}

// the lane's 16 dimensions of the query row ([16 * l8, 16 * l8 + 16)), widened and scaled
__device__ __forceinline__ void q8_load_q(const unsigned char* qrow, int l8, float scale_log2, float2 (&q)[8]) {
  const uint4* qs = reinterpret_cast<const uint4*>(qrow) + 2 * l8;
  const uint4 qa = qs[0], qb = qs[1];
  const float2 sc = make_float2(scale_log2, scale_log2);
  q[0] = __fmul2_rn(widen2(qa.x), sc); q[1] = __fmul2_rn(widen2(qa.y), sc);
  q[2] = __fmul2_rn(widen2(qa.z), sc); q[3] = __fmul2_rn(widen2(qa.w), sc);
  q[4] = __fmul2_rn(widen2(qb.x), sc); q[5] = __fmul2_rn(widen2(qb.y), sc);
  q[6] = __fmul2_rn(widen2(qb.z), sc); q[7] = __fmul2_rn(widen2(qb.w), sc);
}

// The newest token: quantise its rows as the caller passed them (lanes 0-15 the K row, 16-31 the V row) and put
// the slot in its place in the stage and in the slab; later steps read what this step attends to.
__device__ __forceinline__ void q8_store_new(unsigned char* in_stage, const unsigned char* new_rows, unsigned char* in_slab,
                                             int lane) {
  const uint4 raw = reinterpret_cast<const uint4*>(new_rows)[lane];
  const float scale = row_scale16(raw);
  const uint2 codes = quantize8(raw, scale);
  reinterpret_cast<uint2*>(in_stage)[lane] = codes;
  reinterpret_cast<uint2*>(in_slab)[lane] = codes;
  if ((lane & 15) == 0) {
    reinterpret_cast<float*>(in_stage + 256)[lane >> 4] = scale;
    reinterpret_cast<float*>(in_slab + 256)[lane >> 4] = scale;
  }
  __syncwarp();
}

// lanes 0..7 write the output row: lane l8 holds dimensions [16 * l8, 16 * l8 + 16)
__device__ __forceinline__ void q8_write_out(unsigned char* out_row, const State& tot, int l8) {
  const float inv = 1.f / tot.l;
  uint4* dst = reinterpret_cast<uint4*>(out_row) + 2 * l8;
  dst[0] = make_uint4(pack_bf16(tot.acc[0], inv), pack_bf16(tot.acc[1], inv), pack_bf16(tot.acc[2], inv),
                      pack_bf16(tot.acc[3], inv));
  dst[1] = make_uint4(pack_bf16(tot.acc[4], inv), pack_bf16(tot.acc[5], inv), pack_bf16(tot.acc[6], inv),
                      pack_bf16(tot.acc[7], inv));
}

// The 272-byte slot format as the one-layer kernel sees it.
// Two shapes.  15 streaming warps and the finisher: 512 threads keep 128 registers each, which stages of 16
// slots fit; this instance is bound by instruction issue, and the extra warps pay on large layers.  11 warps
// (384 threads, 168 registers) with stages of 24 slots: fewer, longer shares, better on small layers.
template <int kWarpsT, int kChunkT>
struct Q8Slots {
  static constexpr int kWarps = kWarpsT, kStages = 2, kChunk = kChunkT;
  static constexpr int kSlot = kQ8SlotBytes;
  static constexpr int kNewBytes = 2 * kRowBytes;     // the newest token's bf16 rows travel behind the query row
  static constexpr bool kScores = false;              // no row-buffer modes in this format
  static_assert(!kScores, "the one-launch step of this format keeps no score rows");
  using Rows = Q8Rows<kChunk / kGroups>;
  static __device__ __forceinline__ void load_q(const unsigned char* qrow, int l8, float scale_log2, float2 (&q)[8]) {
    q8_load_q(qrow, l8, scale_log2, q);
  }
  static __device__ __forceinline__ void load_stage(const unsigned char* sb, int n, int grp, int l8, Rows& r) {
    q8_load_stage(sb, n, grp, l8, r);
  }
  static __device__ __forceinline__ void fold_stage(const Rows& r, int n, int grp, int, const float2 (&q)[8], State& st,
                                                    const LogitSink&) {
    q8_fold_stage(r, n, grp, q, st);
  }
  static __device__ __forceinline__ void store_new(unsigned char* in_stage, const unsigned char* new_rows,
                                                   unsigned char* in_slab, int lane) {
    q8_store_new(in_stage, new_rows, in_slab, lane);
  }
  static __device__ __forceinline__ void post_acc(float* acc128, const State& tot, int l8) {
    float4* d = reinterpret_cast<float4*>(acc128 + 16 * l8);
#pragma unroll
    for (int j = 0; j < 4; ++j) d[j] = make_float4(tot.acc[2 * j].x, tot.acc[2 * j].y, tot.acc[2 * j + 1].x, tot.acc[2 * j + 1].y);
  }
  static __device__ __forceinline__ void write_out(__nv_bfloat16* out, const State& tot, int l8) {
    q8_write_out(reinterpret_cast<unsigned char*>(out), tot, l8);
  }
};


}  // namespace

cudaError_t launch_quantize_rows(const void* rows, long long n_rows, void* codes, float* scales, cudaStream_t st) {
  const long long threads = n_rows * 16;
  ssd_quantize_rows_kernel<<<(unsigned)((threads + 255) / 256), 256, 0, st>>>(static_cast<const uint4*>(rows), n_rows,
                                                                               static_cast<uint2*>(codes), scales);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_gather_q8(const GatherParams& p, int max_slots, cudaStream_t st) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(p.n_seqs * p.H, (max_slots + 63) / 64 + 1);
  cfg.blockDim = dim3(256);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];                     // behind the selection kernel only (see launch_gather)
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = p.after_select ? 1 : 0;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, ssd_gather_q8_kernel, p);
  count_launch();
  return e;
}

cudaError_t launch_decode_layers_q8(const DecodeLayersParams& p, cudaStream_t st) {
  return launch_decode_step_format<Q8Slots<SSD_Q8_WARPS, SSD_Q8_CHUNK>>(p, st);
}

cudaError_t launch_decode_q8(const DecodeParams& p, cudaStream_t st) {
  // measured per-layer steps, ms (15 x 16 against 11 x 24): 308736 slots per layer 0.695 / 0.724, 209920 slots
  // 0.553 / 0.565, 71680 slots 0.288 / 0.275
  const long total = (long)p.view.cum[p.view.H] * p.view.n_seqs;
  return total >= 131072 ? launch_decode_format<Q8Slots<15, 16>>(p, st) : launch_decode_format<Q8Slots<11, 24>>(p, st);
}

int q8_slot_bytes() { return kQ8SlotBytes; }

}  // namespace ssd
