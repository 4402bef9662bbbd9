// One-time compression of a layer (Algorithm 1, semantic branch; Algorithm 2's prefill split),
// the parts that are not a contraction:
//   select : top-M of score over candidates [0, n0 - R), ties to the lowest index, ascending
//   gather : copy prompt rows, selected rows and the newest ring rows into the slab
// The scores themselves (QK^T, softmax, column sums) come from the tensor-core kernel.
#include "ssd_internal.cuh"

namespace ssd {

namespace {

constexpr int kThreads = 256;

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
