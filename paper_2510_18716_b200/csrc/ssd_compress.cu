// One-time compression of a layer (Algorithm 1, semantic branch; Algorithm 2's prefill split):
//   score  : score[j] = sum over observed image steps t of softmax(q_t K^T)[L + j]   (causal)
//   select : top-M of score over candidates [0, n0 - R), ties to the lowest index, ascending
//   gather : copy prompt rows, selected rows and the newest ring rows into the slab
//
// This file holds the CUDA-core (fp32 FMA) form of the QK^T tiles: every product of two bf16
// values is exact in fp32 and sums are taken in a fixed order, so scores are reproducible bit
// for bit from run to run, which the selection relies on.
#include "ssd_internal.cuh"

namespace ssd {

namespace {

constexpr int kThreads = 256;
constexpr int kBR = 32;        // query rows per block (4 per warp)
constexpr int kBK = 64;        // keys per tile (2 per lane)
constexpr int kKStride = 65;   // padded row stride of the key tile in 32-bit words
constexpr float kNegBig = -1.0e30f;

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float lo_f(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float hi_f(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

struct TileSmem {
  uint32_t k[kBK * kKStride];   // key tile, bf16 pairs
  float2 q[kBR * 64];           // query rows, pre-scaled by scale*log2(e)
};

// rows [r0, r0 + kBR) of Q (n_rows total) -> smem, scaled
__device__ __forceinline__ void load_q_tile(TileSmem& sm, const __nv_bfloat16* Q, int r0, int n_rows,
                                            float scale_log2) {
  const uint32_t* Qw = reinterpret_cast<const uint32_t*>(Q);
  for (int i = threadIdx.x; i < kBR * 64; i += kThreads) {
    int r = i >> 6, dw = i & 63;
    uint32_t w = (r0 + r < n_rows) ? Qw[(size_t)(r0 + r) * 64 + dw] : 0u;
    sm.q[i] = make_float2(lo_f(w) * scale_log2, hi_f(w) * scale_log2);
  }
}

// keys [k0, k0 + kBK) of K (n_keys total) -> smem (zero beyond n_keys)
__device__ __forceinline__ void load_k_tile(TileSmem& sm, const __nv_bfloat16* K, int k0, int n_keys) {
  const uint4* K4 = reinterpret_cast<const uint4*>(K);
  for (int i = threadIdx.x; i < kBK * 16; i += kThreads) {
    int key = i >> 4, c = i & 15;
    uint4 v = (k0 + key < n_keys) ? K4[(size_t)(k0 + key) * 16 + c] : make_uint4(0, 0, 0, 0);
    uint32_t* d = sm.k + key * kKStride + c * 4;
    d[0] = v.x; d[1] = v.y; d[2] = v.z; d[3] = v.w;
  }
}

// logits (base-2 units) of this warp's 4 rows against keys `lane` and `lane + 32` of the tile
__device__ __forceinline__ void tile_logits(const TileSmem& sm, int warp, int lane, float (&x)[4][2]) {
#pragma unroll
  for (int r = 0; r < 4; ++r) x[r][0] = x[r][1] = 0.f;
  const uint32_t* ka = sm.k + lane * kKStride;
  const uint32_t* kb = sm.k + (lane + 32) * kKStride;
  const float2* qr = sm.q + warp * 4 * 64;
#pragma unroll 8
  for (int dw = 0; dw < 64; ++dw) {
    uint32_t a = ka[dw], b = kb[dw];
    float al = lo_f(a), ah = hi_f(a), bl = lo_f(b), bh = hi_f(b);
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      float2 qv = qr[r * 64 + dw];
      x[r][0] = fmaf(al, qv.x, x[r][0]);
      x[r][0] = fmaf(ah, qv.y, x[r][0]);
      x[r][1] = fmaf(bl, qv.x, x[r][1]);
      x[r][1] = fmaf(bh, qv.y, x[r][1]);
    }
  }
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// ----------------------------------------------------------------------------- score
// One CTA per (sequence, semantic head); loops over blocks of 32 observed queries, two passes
// over the key tiles per block (row max / row sum, then normalised column sums).
__global__ void __launch_bounds__(kThreads) ssd_score_kernel(const ScoreParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  TileSmem& sm = *reinterpret_cast<TileSmem*>(smem_raw);
  float* s_part = reinterpret_cast<float*>(smem_raw + sizeof(TileSmem));  // [8][kBK]
  float* s_score = s_part + 8 * kBK;                                      // [n0]

  const int pair = blockIdx.x;
  const int head = pair % p.H;
  if (!p.desc[head].w) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int ctx_all = p.L + p.n0;
  const __nv_bfloat16* Q = p.q_obs + (size_t)pair * p.n_obs * kHeadDim;
  const __nv_bfloat16* K = p.k_full + (size_t)pair * ctx_all * kHeadDim;

  for (int j = tid; j < p.n0; j += kThreads) s_score[j] = 0.f;
  __syncthreads();

  const int t_first = p.n0 - p.n_obs + 1;  // image step of observed row 0
  for (int r0 = 0; r0 < p.n_obs; r0 += kBR) {
    load_q_tile(sm, Q, r0, p.n_obs, p.scale_log2);
    const int rows_here = min(kBR, p.n_obs - r0);
    const int ctx_max = p.L + t_first + r0 + rows_here - 1;  // context of the block's last row
    int ctx_r[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      int row = r0 + warp * 4 + r;
      ctx_r[r] = row < p.n_obs ? p.L + t_first + row : 0;    // keys [0, ctx_r) are visible
    }
    float m[4], s[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) { m[r] = kNegBig; s[r] = 0.f; }

    // pass 1: row max and row sum
    for (int k0 = 0; k0 < ctx_max; k0 += kBK) {
      __syncthreads();
      load_k_tile(sm, K, k0, ctx_all);
      __syncthreads();
      float x[4][2];
      tile_logits(sm, warp, lane, x);
#pragma unroll
      for (int r = 0; r < 4; ++r) {
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          int key = k0 + lane + 32 * c;
          if (key < ctx_r[r]) {
            float mn = fmaxf(m[r], x[r][c]);
            s[r] = s[r] * ex2(m[r] - mn) + ex2(x[r][c] - mn);
            m[r] = mn;
          }
        }
      }
    }
    float inv[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      float mw = warp_max(m[r]);
      float sw = warp_sum(s[r] * ex2(m[r] - mw));
      m[r] = mw;
      inv[r] = sw > 0.f ? 1.f / sw : 0.f;
    }

    // pass 2: normalised probabilities, column sums over the block's rows in a fixed order
    for (int k0 = 0; k0 < ctx_max; k0 += kBK) {
      __syncthreads();
      load_k_tile(sm, K, k0, ctx_all);
      __syncthreads();
      float x[4][2];
      tile_logits(sm, warp, lane, x);
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        int key = k0 + lane + 32 * c;
        float col = 0.f;
#pragma unroll
        for (int r = 0; r < 4; ++r)
          if (key < ctx_r[r]) col += ex2(x[r][c] - m[r]) * inv[r];
        s_part[warp * kBK + lane + 32 * c] = col;
      }
      __syncthreads();
      if (tid < kBK) {
        int key = k0 + tid;
        if (key >= p.L && key < ctx_max) {
          float tot = 0.f;
#pragma unroll
          for (int w = 0; w < 8; ++w) tot += s_part[w * kBK + tid];
          s_score[key - p.L] += tot;
        }
      }
    }
    __syncthreads();
  }
  float* out = p.score + (size_t)pair * p.n0;
  for (int j = tid; j < p.n0; j += kThreads) out[j] = s_score[j];
}

// ----------------------------------------------------------------------------- select
// One CTA per (sequence, semantic head): radix-select the k-th largest score (scores are
// non-negative floats, so their bit patterns order like unsigned integers), then emit, in
// ascending index order, every candidate above it and the lowest-index candidates equal to it.
__global__ void __launch_bounds__(kThreads) ssd_select_kernel(const SelectParams p) {
  __shared__ uint32_t s_hist[256];
  __shared__ uint32_t s_prefix, s_need;
  __shared__ uint32_t s_gt[kThreads + 1], s_eq[kThreads + 1];
  const int pair = blockIdx.x;
  const int head = pair % p.H;
  if (!p.desc[head].w) return;
  const int tid = threadIdx.x;
  const uint32_t* sc = reinterpret_cast<const uint32_t*>(p.score + (size_t)pair * p.n0);
  int32_t* out = p.static_idx + (size_t)pair * p.M;
  const int n = p.n_cand;
  const int k = min(p.M, n);
  for (int i = tid; i < p.M; i += kThreads) out[i] = -1;
  if (k <= 0) return;
  __syncthreads();

  // find the bit pattern of the k-th largest candidate
  if (tid == 0) { s_prefix = 0u; s_need = (uint32_t)k; }
  for (int shift = 24; shift >= 0; shift -= 8) {
    s_hist[tid] = 0u;
    __syncthreads();
    const uint32_t prefix = s_prefix;
    const uint32_t mask = shift == 24 ? 0u : (0xffffffffu << (shift + 8));
    for (int i = tid; i < n; i += kThreads) {
      uint32_t b = sc[i];
      if ((b & mask) == prefix) atomicAdd(&s_hist[(b >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (tid == 0) {
      uint32_t need = s_need, cum = 0u;
      int bin = 255;
      for (; bin > 0; --bin) {
        if (cum + s_hist[bin] >= need) break;
        cum += s_hist[bin];
      }
      s_need = need - cum;
      s_prefix = prefix | ((uint32_t)bin << shift);
    }
    __syncthreads();
  }
  const uint32_t thr = s_prefix;      // k-th largest value
  const uint32_t need_eq = s_need;    // how many candidates equal to it are taken (lowest index)

  // ordered compaction: each thread owns a contiguous segment of candidates
  const int seg = (n + kThreads - 1) / kThreads;
  const int a = min(n, tid * seg), b = min(n, a + seg);
  uint32_t cg = 0u, ce = 0u;
  for (int i = a; i < b; ++i) {
    uint32_t v = sc[i];
    cg += v > thr;
    ce += v == thr;
  }
  s_gt[tid + 1] = cg;
  s_eq[tid + 1] = ce;
  if (tid == 0) { s_gt[0] = 0u; s_eq[0] = 0u; }
  __syncthreads();
  if (tid == 0) {
    for (int i = 1; i <= kThreads; ++i) {
      s_gt[i] += s_gt[i - 1];
      s_eq[i] += s_eq[i - 1];
    }
  }
  __syncthreads();
  uint32_t g_before = s_gt[tid], e_before = s_eq[tid];
  for (int i = a; i < b; ++i) {
    uint32_t v = sc[i];
    if (v > thr) {
      out[g_before + min(e_before, need_eq)] = i;
      ++g_before;
    } else if (v == thr) {
      if (e_before < need_eq) out[g_before + e_before] = i;
      ++e_before;
    }
  }
}

// ----------------------------------------------------------------------------- gather
// One warp per destination slot: lanes 0-15 copy the K row, lanes 16-31 the V row.
__global__ void __launch_bounds__(kThreads) ssd_gather_kernel(const GatherParams p, int max_slots) {
  const int pair = blockIdx.x;
  const int seq = pair / p.H, head = pair - seq * p.H;
  const HeadDesc d = p.desc[head];
  const int cap = p.L + d.y + d.z;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int ctx = p.L + p.n0;
  uint4* dst0 = p.slab + ((size_t)seq * p.seq_slots + d.x) * kSlotU4;
  const uint4* src = (lane < 16 ? p.k_full : p.v_full) + (size_t)pair * ctx * 16 + (lane & 15);
  for (int s = blockIdx.y * 8 + warp; s < cap; s += gridDim.y * 8) {
    int pos = -1;
    if (s < p.L) {
      pos = s;
    } else if (s < p.L + d.y) {
      int mm = s - p.L;
      if (d.w && mm < p.static_valid) {
        int j = p.static_idx[(size_t)pair * p.M + mm];
        if (j >= 0 && j < p.n0) pos = p.L + j;
      }
    } else {
      int r = s - p.L - d.y;                       // ring slot r holds the newest j = r (mod cap)
      if (p.n0 - 1 >= r) pos = p.L + ((p.n0 - 1 - r) / d.z) * d.z + r;
    }
    if (pos >= 0) dst0[(size_t)s * kSlotU4 + lane] = src[(size_t)pos * 16];
  }
}

}  // namespace

cudaError_t launch_score(const ScoreParams& p, cudaStream_t st) {
  size_t smem = sizeof(TileSmem) + (8 * kBK + (size_t)p.n0) * sizeof(float);
  cudaError_t e = cudaFuncSetAttribute(ssd_score_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  ssd_score_kernel<<<p.n_seqs * p.H, kThreads, smem, st>>>(p);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_select(const SelectParams& p, cudaStream_t st) {
  ssd_select_kernel<<<p.n_seqs * p.H, kThreads, 0, st>>>(p);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_gather(const GatherParams& p, int max_slots, cudaStream_t st) {
  dim3 grid(p.n_seqs * p.H, (max_slots + 63) / 64);
  ssd_gather_kernel<<<grid, kThreads, 0, st>>>(p, max_slots);
  count_launch();
  return cudaGetLastError();
}

}  // namespace ssd
