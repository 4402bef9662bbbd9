// Single-token decode attention over the head-decoupled compressed KV store, and the
// per-step append/evict.
//
// Decode (consumer of Algorithm 1's output): for every (sequence, head) of one layer,
//   out = sum_i softmax_i(scale * <q, K_i>) V_i   over the slots that hold a token.
// It is a GEMV per head (1 flop per byte), so the kernel is built around HBM streaming, not
// tensor cores:
//   * the valid slots of the whole layer form one logical stream of 512-byte slots
//     ([K row | V row]); the stream is cut into equal, 8-slot-aligned shares, one per warp
//     ("worker"), regardless of head type or length, so every SM gets the same bytes;
//   * a worker walks its share pair by pair; half-warp 0/1 take even/odd slots, 16 lanes x
//     128-bit loads cover one row; dot products are reduced with shuffles inside the
//     half-warp; online softmax in fp32 (base-2 exponent, scale folded into q);
//   * a pair that lies inside one share is finished in registers; a pair cut by a share
//     boundary leaves (m, l, acc[128]) partials in scratch and the last contributor to
//     arrive (atomic counter, never waits) merges them in worker order, which keeps the
//     result independent of arrival order.
#include "ssd_internal.cuh"

namespace ssd {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kCtasPerSm = 3;
constexpr int kU = 4;               // slots per half-warp per iteration
constexpr int kAlign = 8;           // share boundaries are multiples of this many slots
constexpr int kMinShare = 16;       // never cut shares smaller than this
constexpr float kNegBig = -1.0e30f;

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
  uint4 v;
  asm("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
      : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
      : "l"(p));
  return v;
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ float lo_f(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float hi_f(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

__device__ __forceinline__ float dot8(const uint4& k, const float (&q)[8]) {
  float a = lo_f(k.x) * q[0];
  a = fmaf(hi_f(k.x), q[1], a);
  a = fmaf(lo_f(k.y), q[2], a);
  a = fmaf(hi_f(k.y), q[3], a);
  a = fmaf(lo_f(k.z), q[4], a);
  a = fmaf(hi_f(k.z), q[5], a);
  a = fmaf(lo_f(k.w), q[6], a);
  a = fmaf(hi_f(k.w), q[7], a);
  return a;
}

__device__ __forceinline__ void axpy8(float p, const uint4& v, float (&acc)[8]) {
  acc[0] = fmaf(p, lo_f(v.x), acc[0]);
  acc[1] = fmaf(p, hi_f(v.x), acc[1]);
  acc[2] = fmaf(p, lo_f(v.y), acc[2]);
  acc[3] = fmaf(p, hi_f(v.y), acc[3]);
  acc[4] = fmaf(p, lo_f(v.z), acc[4]);
  acc[5] = fmaf(p, hi_f(v.z), acc[5]);
  acc[6] = fmaf(p, lo_f(v.w), acc[6]);
  acc[7] = fmaf(p, hi_f(v.w), acc[7]);
}

struct State {
  float m, l;
  float acc[8];
};

__device__ __forceinline__ void state_init(State& s) {
  s.m = kNegBig;
  s.l = 0.f;
#pragma unroll
  for (int d = 0; d < 8; ++d) s.acc[d] = 0.f;
}

// s <- s (+) (m2, l2, acc2)
__device__ __forceinline__ void state_merge(State& s, float m2, float l2, const float (&a2)[8]) {
  float mn = fmaxf(s.m, m2);
  float c1 = ex2(s.m - mn), c2 = ex2(m2 - mn);
  s.l = s.l * c1 + l2 * c2;
#pragma unroll
  for (int d = 0; d < 8; ++d) s.acc[d] = s.acc[d] * c1 + a2[d] * c2;
  s.m = mn;
}

// Stream `n` physically contiguous slots starting at `base` into the running state of this
// half-warp (hw = 0/1 takes even/odd slots).
__device__ __forceinline__ void process_piece(const uint4* __restrict__ base, int n, int hw, int l16,
                                              const float (&q)[8], State& st) {
  for (int s = 0; s < n; s += 2 * kU) {
    uint4 k[kU], v[kU];
    bool ok[kU];
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      int slot = s + 2 * u + hw;
      ok[u] = slot < n;
      const uint4* p = base + (size_t)slot * kSlotU4 + l16;
      if (ok[u]) {
        k[u] = ld_stream(p);
        v[u] = ld_stream(p + 16);
      } else {
        k[u] = make_uint4(0, 0, 0, 0);
        v[u] = make_uint4(0, 0, 0, 0);
      }
    }
    float x[kU];
#pragma unroll
    for (int u = 0; u < kU; ++u) x[u] = dot8(k[u], q);
#pragma unroll
    for (int off = 8; off >= 1; off >>= 1) {
#pragma unroll
      for (int u = 0; u < kU; ++u) x[u] += __shfl_xor_sync(0xffffffffu, x[u], off);
    }
    float mn = st.m;
#pragma unroll
    for (int u = 0; u < kU; ++u) mn = fmaxf(mn, ok[u] ? x[u] : kNegBig);
    float corr = ex2(st.m - mn);
    float p[kU], psum = 0.f;
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      p[u] = ok[u] ? ex2(x[u] - mn) : 0.f;
      psum += p[u];
    }
    st.l = st.l * corr + psum;
    st.m = mn;
#pragma unroll
    for (int d = 0; d < 8; ++d) st.acc[d] *= corr;
#pragma unroll
    for (int u = 0; u < kU; ++u) axpy8(p[u], v[u], st.acc);
  }
}

__device__ __forceinline__ long share_start(long i, long T, long W) {
  if (i >= W) return T;
  return ((i * T) / W) & ~(long)(kAlign - 1);
}

// Largest worker index whose share starts at or before logical slot g.
__device__ __forceinline__ long share_of(long g, long T, long W) {
  long gp = (g & ~(long)(kAlign - 1)) + kAlign;
  long w = (gp * W - 1) / T;
  return w < W - 1 ? w : W - 1;
}

__device__ __forceinline__ void write_out(__nv_bfloat16* out, const State& st, int l16) {
  float inv = 1.f / st.l;
  uint4 o;
  __nv_bfloat162 t;
  t = __floats2bfloat162_rn(st.acc[0] * inv, st.acc[1] * inv);
  o.x = *reinterpret_cast<uint32_t*>(&t);
  t = __floats2bfloat162_rn(st.acc[2] * inv, st.acc[3] * inv);
  o.y = *reinterpret_cast<uint32_t*>(&t);
  t = __floats2bfloat162_rn(st.acc[4] * inv, st.acc[5] * inv);
  o.z = *reinterpret_cast<uint32_t*>(&t);
  t = __floats2bfloat162_rn(st.acc[6] * inv, st.acc[7] * inv);
  o.w = *reinterpret_cast<uint32_t*>(&t);
  reinterpret_cast<uint4*>(out)[l16] = o;
}

__global__ void __launch_bounds__(kThreads, kCtasPerSm) decode_kernel(const DecodeParams p) {
  __shared__ int s_cum[kMaxHeads + 1];  // exclusive prefix of valid slots per head
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int hw = lane >> 4, l16 = lane & 15;

  // valid slots per head, then an exclusive scan by warp 0 (4 heads per lane)
  if (tid < 32) {
    int v[4], sum = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int h = tid * 4 + i;
      v[i] = 0;
      if (h < p.H) {
        HeadDesc d = p.desc[h];
        v[i] = p.prompt_valid + (d.w ? p.static_valid : 0) + min(p.t_img, d.z);
      }
      sum += v[i];
    }
    int incl = sum;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      int o = __shfl_up_sync(0xffffffffu, incl, off);
      if (tid >= off) incl += o;
    }
    int run = incl - sum;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int h = tid * 4 + i;
      if (h <= p.H) s_cum[h] = run;
      run += v[i];
    }
    if (tid == 31 && p.H == kMaxHeads) s_cum[kMaxHeads] = run;
  }
  __syncthreads();

  const long Vseq = s_cum[p.H];
  const long T = Vseq * p.n_seqs;
  const long W = p.n_workers;
  const long wk = (long)blockIdx.x * kWarps + warp;
  if (wk >= W) return;

  long g = share_start(wk, T, W);
  const long g_end = share_start(wk + 1, T, W);
  bool first = true;

  while (g < g_end) {
    const int seq = (int)(g / Vseq);
    const int r = (int)(g - (long)seq * Vseq);
    int lo = 0, hi = p.H;  // find head with s_cum[head] <= r < s_cum[head+1]
    while (hi - lo > 1) {
      int mid = (lo + hi) >> 1;
      if (s_cum[mid] <= r) lo = mid; else hi = mid;
    }
    const int head = lo;
    const int vh = s_cum[head + 1] - s_cum[head];
    const int i0 = r - s_cum[head];
    const long left = g_end - g;
    const int i1 = (long)(vh - i0) <= left ? vh : i0 + (int)left;

    const HeadDesc d = p.desc[head];
    const int pair = seq * p.H + head;
    const uint4* pbase = p.slab + ((size_t)seq * p.seq_slots + d.x) * kSlotU4;

    float q[8];
    {
      uint4 qq = reinterpret_cast<const uint4*>(p.q + (size_t)pair * kHeadDim)[l16];
      q[0] = lo_f(qq.x) * p.scale_log2; q[1] = hi_f(qq.x) * p.scale_log2;
      q[2] = lo_f(qq.y) * p.scale_log2; q[3] = hi_f(qq.y) * p.scale_log2;
      q[4] = lo_f(qq.z) * p.scale_log2; q[5] = hi_f(qq.z) * p.scale_log2;
      q[6] = lo_f(qq.w) * p.scale_log2; q[7] = hi_f(qq.w) * p.scale_log2;
    }
    State st;
    state_init(st);

    // three physically contiguous runs: prompt, static, ring
    const int sv = d.w ? p.static_valid : 0;
    const int rv = min(p.t_img, d.z);
    const int run_l0[3] = {0, p.prompt_valid, p.prompt_valid + sv};
    const int run_n[3] = {p.prompt_valid, sv, rv};
    const int run_p0[3] = {0, p.L, p.L + d.y};
#pragma unroll
    for (int rr = 0; rr < 3; ++rr) {
      int a = max(i0, run_l0[rr]);
      int b = min(i1, run_l0[rr] + run_n[rr]);
      if (b > a)
        process_piece(pbase + (size_t)(run_p0[rr] + (a - run_l0[rr])) * kSlotU4, b - a, hw, l16, q, st);
    }

    // merge the two half-warps (lanes i and i+16 hold the same 8 output dims)
    {
      float m2 = __shfl_xor_sync(0xffffffffu, st.m, 16);
      float l2 = __shfl_xor_sync(0xffffffffu, st.l, 16);
      float a2[8];
#pragma unroll
      for (int dd = 0; dd < 8; ++dd) a2[dd] = __shfl_xor_sync(0xffffffffu, st.acc[dd], 16);
      state_merge(st, m2, l2, a2);
    }

    __nv_bfloat16* outp = p.out + (size_t)pair * kHeadDim;
    if (i0 == 0 && i1 == vh) {
      if (hw == 0) write_out(outp, st, l16);
    } else {
      float* P = p.partial + ((size_t)wk * 2 + (first ? 0 : 1)) * kPartialFloats;
      if (lane == 0) {
        P[0] = st.m;
        P[1] = st.l;
      }
      if (hw == 0) {
        reinterpret_cast<float4*>(P + 4)[l16 * 2] = make_float4(st.acc[0], st.acc[1], st.acc[2], st.acc[3]);
        reinterpret_cast<float4*>(P + 4)[l16 * 2 + 1] = make_float4(st.acc[4], st.acc[5], st.acc[6], st.acc[7]);
      }
      __threadfence();
      __syncwarp();
      const long g0 = g - i0, g1 = g0 + vh;
      const long w_lo = share_of(g0, T, W), w_hi = share_of(g1 - 1, T, W);
      const uint32_t n_contrib = (uint32_t)(w_hi - w_lo + 1);
      uint32_t old = 0;
      if (lane == 0) old = atomicAdd(p.counters + pair, 1u);
      old = __shfl_sync(0xffffffffu, old, 0);
      if (old == n_contrib - 1) {
        __threadfence();
        State tot;
        state_init(tot);
        for (long j = w_lo; j <= w_hi; ++j) {
          int which = (j == w_lo && share_start(j, T, W) < g0) ? 1 : 0;
          const float* Pj = p.partial + ((size_t)j * 2 + which) * kPartialFloats;
          float mj = __ldcg(Pj), lj = __ldcg(Pj + 1);
          float4 x0 = __ldcg(reinterpret_cast<const float4*>(Pj + 4) + l16 * 2);
          float4 x1 = __ldcg(reinterpret_cast<const float4*>(Pj + 4) + l16 * 2 + 1);
          float aj[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
          state_merge(tot, mj, lj, aj);
        }
        if (hw == 0) write_out(outp, tot, l16);
        if (lane == 0) p.counters[pair] = 0u;
      }
    }
    g += i1 - i0;
    first = false;
  }
}

__global__ void __launch_bounds__(256) append_kernel(const AppendParams p) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= p.n_seqs * p.H) return;
  const int seq = warp / p.H, head = warp - seq * p.H;
  const HeadDesc d = p.desc[head];
  const int ring_slot = p.j % d.z;
  uint4* dst = p.slab + ((size_t)seq * p.seq_slots + d.x + p.L + d.y + ring_slot) * kSlotU4;
  const uint4* src = (lane < 16 ? p.k_new : p.v_new) + (size_t)warp * 16 + (lane & 15);
  dst[lane] = *src;
}

}  // namespace

int decode_max_workers() {
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) {
    int v = 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0) sms = v;
  }
  if (sms < 148) sms = 148;  // size scratch for at least a full B200
  return sms * kCtasPerSm * kWarps;
}

cudaError_t launch_decode(const DecodeParams& p_in, long total_valid, cudaStream_t st) {
  DecodeParams p = p_in;
  long w = decode_max_workers();
  long cap = total_valid / kMinShare;
  if (cap < 1) cap = 1;
  if (w > cap) w = cap;
  p.n_workers = (int)w;
  int grid = (int)((w + kWarps - 1) / kWarps);
  decode_kernel<<<grid, kThreads, 0, st>>>(p);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_append(const AppendParams& p, cudaStream_t st) {
  int warps = p.n_seqs * p.H;
  int grid = (warps * 32 + 255) / 256;
  append_kernel<<<grid, 256, 0, st>>>(p);
  count_launch();
  return cudaGetLastError();
}

}  // namespace ssd
