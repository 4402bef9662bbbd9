// One-time compression of a layer (Algorithm 1, semantic branch; Algorithm 2's prefill split),
// the parts that are not a contraction:
//   select : top-M of score over candidates [0, n0 - R), ties to the lowest index, ascending
//   gather : copy prompt rows, selected rows and the newest ring rows into the slab
// The scores themselves (QK^T, softmax, column sums) come from the tensor-core kernel.
#include "ssd_internal.cuh"

namespace ssd {

namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
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
  float* acc = p.acc ? p.acc + (size_t)pair * p.mr : nullptr;   // row-buffer mode: scores travel with the tokens
  for (int i = a; i < b; ++i) {
    uint32_t v = sc[i];
    if (v > thr) {
      const uint32_t o = g_before + min(e_before, need_eq);
      out[o] = i;
      if (acc) acc[o] = __uint_as_float(v);
      ++g_before;
    } else if (v == thr) {
      if (e_before < need_eq) {
        out[g_before + e_before] = i;
        if (acc) acc[g_before + e_before] = __uint_as_float(v);
      }
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
      if (p.n0 - 1 >= r && (p.sem_ring || !d.w)) pos = p.L + ((p.n0 - 1 - r) / d.z) * d.z + r;
    }
    if (pos >= 0) dst0[(size_t)s * kSlotU4 + lane] = src[(size_t)pos * 16];
  }
}

// ----------------------------------------------------------------------------- recompress
// Algorithm 2, "row buffer full": for every (sequence, semantic head) keep the top-M of the static
// set plus the buffered tokens by accumulated attention score (ties: lowest position), in ascending
// position, as the new static set; the buffer is then empty.  One CTA per pair.  Candidates are
// already in ascending position (static slots, then buffer slots), so selection is an ordered
// compaction, done in place: a kept row never moves to a higher slot, and rows are moved through
// shared memory in ascending batches, so no source is overwritten before it is read.
constexpr int kMoveBatch = 32;

__device__ __forceinline__ void recompress_pair(const RecompressParams& p, int pair) {
  extern __shared__ __align__(16) unsigned char rsm[];
  __shared__ uint32_t s_hist[256];
  __shared__ uint32_t s_prefix, s_need;
  __shared__ int s_count;
  const int seq = pair / p.H, head = pair - seq * p.H;
  const HeadDesc d = p.desc[head];
  if (!d.w) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n = p.static_valid + p.buffered;          // candidates
  const int k = min(p.M, n);
  float* s_sc = reinterpret_cast<float*>(rsm);         // [mr] candidate scores, candidate order
  int* s_pos = reinterpret_cast<int*>(s_sc + p.mr);    // [mr] candidate image indices
  int* s_keep = s_pos + p.mr;                          // [mr] kept candidates, ascending
  uint4* s_rows = reinterpret_cast<uint4*>(s_keep + p.mr + ((4 - (3 * p.mr) % 4) % 4));   // [kMoveBatch][32]
  float* acc = p.acc + (size_t)pair * p.mr;
  int32_t* idx = p.static_idx + (size_t)pair * p.M;

  // candidate c lives in entry e(c) of the score row and of the head's static+ring slots
  for (int c = tid; c < n; c += kThreads) {
    const int e = c < p.static_valid ? c : d.y + (c - p.static_valid);
    float sc = acc[e];
    if (p.pending) {
      const float2 ml = p.ml[pair];
      sc += ex2(p.logits[(size_t)pair * p.mr + e] - ml.x) / ml.y;
    }
    s_sc[c] = sc;
    s_pos[c] = c < p.static_valid ? idx[c] : p.t_base + (c - p.static_valid);
  }
  __syncthreads();

  // bit pattern of the k-th largest score (scores are non-negative)
  const uint32_t* bits = reinterpret_cast<const uint32_t*>(s_sc);
  if (tid == 0) { s_prefix = 0u; s_need = (uint32_t)k; s_count = 0; }
  for (int shift = 24; shift >= 0; shift -= 8) {
    s_hist[tid] = 0u;
    __syncthreads();
    const uint32_t prefix = s_prefix;
    const uint32_t mask = shift == 24 ? 0u : (0xffffffffu << (shift + 8));
    for (int i = tid; i < n; i += kThreads) {
      const uint32_t b = bits[i];
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
  // ordered compaction by one warp: above the threshold, or equal to it among the first s_need such
  if (warp == 0) {
    const uint32_t thr = s_prefix;
    uint32_t eq_left = s_need;
    int kept = 0;
    for (int c0 = 0; c0 < n; c0 += 32) {
      const int c = c0 + lane;
      const uint32_t b = c < n ? bits[c] : 0u;
      const bool gt = c < n && b > thr, eq = c < n && b == thr;
      const unsigned eq_mask = __ballot_sync(0xffffffffu, eq);
      const uint32_t eq_before = __popc(eq_mask & ((1u << lane) - 1u));
      const bool take = gt || (eq && eq_before < eq_left);
      const unsigned take_mask = __ballot_sync(0xffffffffu, take);
      if (take) s_keep[kept + __popc(take_mask & ((1u << lane) - 1u))] = c;
      kept += __popc(take_mask);
      const uint32_t eq_taken = min((uint32_t)__popc(eq_mask), eq_left);
      eq_left -= eq_taken;
    }
    if (lane == 0) s_count = kept;
  }
  __syncthreads();
  const int kept = s_count;                            // == k

  // scores and positions of the new static set
  float my_sc[2];
  int my_pos[2];
  for (int r = 0; r < 2; ++r) {
    const int o = tid + r * kThreads;
    if (o < kept) { my_sc[r] = s_sc[s_keep[o]]; my_pos[r] = s_pos[s_keep[o]]; }
  }
  // rows: slot of candidate c is L + e(c); destination of the o-th kept row is static slot o
  uint4* hbase = p.slab + ((size_t)seq * p.seq_slots + d.x + p.L) * kSlotU4;
  for (int o0 = 0; o0 < kept; o0 += kMoveBatch) {
    const int nb = min(kMoveBatch, kept - o0);
    // a kept static row that no dropped row precedes is already where it belongs (candidate c of the
    // static set sits in slot c): neither read nor written
    for (int r = warp; r < nb; r += kThreads / 32) {
      const int c = s_keep[o0 + r];
      if (c == o0 + r) continue;
      const int e = c < p.static_valid ? c : d.y + (c - p.static_valid);
      s_rows[r * 32 + lane] = hbase[(size_t)e * kSlotU4 + lane];
    }
    __syncthreads();
    for (int r = warp; r < nb; r += kThreads / 32)
      if (s_keep[o0 + r] != o0 + r) hbase[(size_t)(o0 + r) * kSlotU4 + lane] = s_rows[r * 32 + lane];
    __syncthreads();
  }
  for (int r = 0; r < 2; ++r) {
    const int o = tid + r * kThreads;
    if (o < kept) { acc[o] = my_sc[r]; idx[o] = my_pos[r]; }
  }
  for (int o = kept + tid; o < p.M; o += kThreads) idx[o] = -1;
}

__global__ void __launch_bounds__(kThreads) ssd_recompress_kernel(const RecompressParams p) { recompress_pair(p, blockIdx.x); }

// One CTA per (pair, layer): blockIdx.y is the layer.
__global__ void __launch_bounds__(kThreads) ssd_recompress_layers_kernel(const __grid_constant__ RecompressLayersParams q) {
  const int layer = blockIdx.y;
  const RecompressLayer& ly = q.layer[layer];
  if (!ly.todo) return;
  const size_t pairs = (size_t)q.n_seqs * q.H;
  RecompressParams p;
  p.slab = q.slab + (size_t)ly.first_slot * kSlotU4;
  p.desc = q.desc + (size_t)layer * q.H;
  p.static_idx = q.static_idx + (size_t)layer * pairs * (q.M > 0 ? q.M : 1);
  p.acc = q.acc + (size_t)layer * pairs * q.mr;
  p.logits = q.logits + (size_t)layer * pairs * q.mr;
  p.ml = q.ml + (size_t)layer * pairs;
  p.pending = ly.pending;
  p.n_seqs = q.n_seqs; p.H = q.H; p.L = q.L; p.M = q.M; p.mr = q.mr;
  p.static_valid = ly.static_valid;
  p.buffered = ly.buffered;
  p.t_base = ly.t_base;
  p.seq_slots = ly.seq_slots;
  recompress_pair(p, blockIdx.x);
}

}  // namespace

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

cudaError_t launch_recompress_layers(const RecompressLayersParams& p, cudaStream_t st) {
  if (p.M > 2 * kThreads || p.n_layers < 1 || p.n_layers > kMaxLayersPerLaunch) return cudaErrorInvalidValue;
  const size_t smem = (size_t)(3 * p.mr + 4) * 4 + (size_t)kMoveBatch * 512;
  cudaError_t e = cudaFuncSetAttribute(ssd_recompress_layers_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  ssd_recompress_layers_kernel<<<dim3(p.n_seqs * p.H, p.n_layers), kThreads, smem, st>>>(p);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_recompress(const RecompressParams& p, cudaStream_t st) {
  if (p.M > 2 * kThreads) return cudaErrorInvalidValue;      // each thread carries two kept entries
  const size_t smem = (size_t)(3 * p.mr + 4) * 4 + (size_t)kMoveBatch * 512;
  cudaError_t e = cudaFuncSetAttribute(ssd_recompress_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  ssd_recompress_kernel<<<p.n_seqs * p.H, kThreads, smem, st>>>(p);
  count_launch();
  return cudaGetLastError();
}

}  // namespace ssd
