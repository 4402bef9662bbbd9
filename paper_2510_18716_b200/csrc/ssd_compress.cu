// One-time compression of a layer (Algorithm 1, semantic branch; Algorithm 2's prefill split),
// the parts that are not a contraction:
//   select : top-M of score over candidates [0, n0 - R), ties to the lowest index, ascending
//   gather : copy prompt rows, selected rows and the newest ring rows into the slab
// The scores themselves (QK^T, softmax, column sums) come from the tensor-core kernel.
#include "ssd_internal.cuh"
#include "ssd_device.cuh"

namespace ssd {

namespace {

constexpr int kThreads = 256;

// Selection among few candidates without a radix pass: candidate c is kept iff fewer than k
// candidates come before it in the order (score descending, then position ascending); its rank is
// counted directly (n * n / kThreads comparisons per thread, all reading the same shared-memory
// word at a time).  bits[]: the scores' bit patterns (non-negative floats order like unsigned
// integers); pos == nullptr means a candidate's position is its index.
constexpr int kRankMax = 1024;

__device__ __forceinline__ void rank_select(const uint32_t* bits, const int* pos, int n, int k, int* flag) {
  for (int c = threadIdx.x; c < n; c += kThreads) {
    const uint32_t b = bits[c];
    const int pc = pos ? pos[c] : c;
    int rank = 0;
    for (int j = 0; j < n; ++j) {
      const uint32_t bj = bits[j];
      const int pj = pos ? pos[j] : j;
      rank += (bj > b || (bj == b && pj < pc)) ? 1 : 0;
    }
    flag[c] = rank < k ? 1 : 0;
  }
}

// Radix-select helpers shared by the selection and the re-selection: one digit of 8 bits per pass.
// hist[b] += candidates of this thread's value with digit b; lanes of a warp that hold the same digit add once
// (scores of one head share their leading digits, so most of a warp lands in one or two bins).
__device__ __forceinline__ void hist_add(uint32_t* hist, bool take, uint32_t digit) {
  const unsigned active = __ballot_sync(0xffffffffu, take);
  if (!take) return;
  const unsigned same = __match_any_sync(active, digit);
  if ((int)(threadIdx.x & 31) == __ffs(same) - 1) atomicAdd(&hist[digit], (uint32_t)__popc(same));
}
// Run by warp 0 after a pass: the highest bin b with (candidates in bins > b) < need <= (candidates in bins >= b);
// returns it and takes the candidates above it off `need`.  Lane l owns bins [8l, 8l + 8).
__device__ __forceinline__ int pick_bin(const uint32_t* hist, uint32_t& need, int lane) {
  uint32_t own[8], t = 0u;
#pragma unroll
  for (int j = 0; j < 8; ++j) { own[j] = hist[8 * lane + j]; t += own[j]; }
  uint32_t incl = t;                                   // sum over lanes >= this one
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const uint32_t o = __shfl_down_sync(0xffffffffu, incl, off);
    if (lane + off < 32) incl += o;
  }
  const unsigned ok = __ballot_sync(0xffffffffu, incl >= need);
  const int owner = ok ? 31 - __clz(ok) : 0;          // (never empty: need <= the candidates that are left)
  int bin = 0;
  uint32_t left = need;
  if (lane == owner) {
    uint32_t cum = incl - t;                           // candidates in the bins of higher lanes
    bin = 8 * lane + 7;
    for (; bin > 8 * lane; --bin) {
      if (cum + own[bin - 8 * lane] >= need) break;
      cum += own[bin - 8 * lane];
    }
    left = need - cum;
  }
  need = __shfl_sync(0xffffffffu, left, owner);
  return __shfl_sync(0xffffffffu, bin, owner);
}
// Exclusive prefix sums over the thread block of two counters per thread (kThreads = 8 warps); s_w: 2 x 8 words.
__device__ __forceinline__ void block_prefix2(uint32_t& a, uint32_t& b, uint32_t (*s_w)[8]) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t ia = a, ib = b;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const uint32_t oa = __shfl_up_sync(0xffffffffu, ia, off), ob = __shfl_up_sync(0xffffffffu, ib, off);
    if (lane >= off) { ia += oa; ib += ob; }
  }
  if (lane == 31) { s_w[0][warp] = ia; s_w[1][warp] = ib; }
  __syncthreads();
  uint32_t ba = 0u, bb = 0u;
  for (int w = 0; w < warp; ++w) { ba += s_w[0][w]; bb += s_w[1][w]; }
  a = ba + ia - a;
  b = bb + ib - b;
}

// ----------------------------------------------------------------------------- select
// One CTA per (sequence, semantic head): radix-select the k-th largest score (scores are
// non-negative floats, so their bit patterns order like unsigned integers), then emit, in
// ascending index order, every candidate above it and the lowest-index candidates equal to it.
__global__ void __launch_bounds__(kThreads) ssd_select_kernel(const SelectParams p) {
  __shared__ uint32_t s_hist[256];
  __shared__ uint32_t s_prefix, s_need;
  __shared__ uint32_t s_scan[2][8];
  const int pair = blockIdx.x;
  const int head = pair % p.H;
  pdl_allow_successor();      // the gather that follows copies what does not depend on this kernel meanwhile
  if (!p.desc[head].w) return;
  const int tid = threadIdx.x;
  // the score row arrives in 2 * n_parts pieces (one per half of the query rows, from every thread block that
  // shared the pair's query blocks): add them in a fixed order, so the row is reproducible bit for bit
  float* row = p.score + (size_t)pair * kScoreHalves * p.n0;
  {
    const size_t stride = (size_t)gridDim.x * kScoreHalves * p.n0;
    for (int i = tid; i < p.n0; i += kThreads) {
      float s = 0.f;
      for (int part = 0; part < p.n_parts; ++part) {
        const float* r = row + (size_t)part * stride + i;
        s += r[0] + r[p.n0];
      }
      row[i] = s;
    }
    __syncthreads();
  }
  const uint32_t* sc = reinterpret_cast<const uint32_t*>(row);
  int32_t* out = p.static_idx + (size_t)pair * p.M;
  const int n = p.n_cand;
  const int k = min(p.M, n);
  for (int i = tid; i < p.M; i += kThreads) out[i] = -1;
  if (k <= 0) return;
  __syncthreads();
  float* acc_row = p.acc ? p.acc + (size_t)pair * p.mr : nullptr;   // row-buffer mode: scores travel with the tokens
  if (n <= kRankMax) {
    __shared__ uint32_t s_bits[kRankMax];
    __shared__ int s_flag[kRankMax];
    for (int i = tid; i < n; i += kThreads) s_bits[i] = sc[i];
    __syncthreads();
    rank_select(s_bits, nullptr, n, k, s_flag);
    __syncthreads();
    if (tid < 32) {                    // ordered compaction by one warp
      int cnt = 0;
      for (int c0 = 0; c0 < n; c0 += 32) {
        const int c = c0 + tid;
        const bool take = c < n && s_flag[c];
        const unsigned m = __ballot_sync(0xffffffffu, take);
        if (take) {
          const int o = cnt + __popc(m & ((1u << tid) - 1u));
          out[o] = c;
          if (acc_row) acc_row[o] = __uint_as_float(s_bits[c]);
        }
        cnt += __popc(m);
      }
    }
    return;
  }

  // find the bit pattern of the k-th largest candidate
  if (tid == 0) { s_prefix = 0u; s_need = (uint32_t)k; }
  for (int shift = 24; shift >= 0; shift -= 8) {
    s_hist[tid] = 0u;
    __syncthreads();
    const uint32_t prefix = s_prefix;
    const uint32_t mask = shift == 24 ? 0u : (0xffffffffu << (shift + 8));
    for (int i0 = 0; i0 < n; i0 += kThreads) {         // every thread takes part in every round (warp votes inside)
      const int i = i0 + tid;
      const uint32_t b = i < n ? sc[i] : 0u;
      hist_add(s_hist, i < n && (b & mask) == prefix, (b >> shift) & 255u);
    }
    __syncthreads();
    if (tid < 32) {
      uint32_t need = s_need;
      const int bin = pick_bin(s_hist, need, tid);
      if (tid == 0) {
        s_need = need;
        s_prefix = prefix | ((uint32_t)bin << shift);
      }
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
  uint32_t g_before = cg, e_before = ce;          // candidates above / equal to the threshold in earlier segments
  block_prefix2(g_before, e_before, s_scan);
  float* acc = acc_row;
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
// One warp per destination slot, two slots at a time (both rows are on their way before the first is stored):
// lanes 0-15 copy the K row, lanes 16-31 the V row.  Thread blocks (pair, y < gridDim.y - 1) share the slots that
// do not depend on the selection (prompt, rings, everything of a spatial head); the blocks of the last y, which
// are handed out after all the others, copy the static slots of semantic heads once the selection kernel has
// completed.  Launched as that kernel's programmatic dependent, everything but those last blocks runs beside it.
__global__ void __launch_bounds__(kThreads) ssd_gather_kernel(const GatherParams p) {
  const int pair = blockIdx.x;
  const int seq = pair / p.H, head = pair - seq * p.H;
  const HeadDesc d = p.desc[head];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int ctx = p.L + p.n0;
  uint4* dst0 = p.slab + ((size_t)seq * p.seq_slots + d.x) * kSlotU4;
  const uint4* src = (lane < 16 ? p.k_full : p.v_full) + (size_t)pair * ctx * 16 + (lane & 15);
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
    const int pa = a ? gather_source_row(p, d, pair, s) : -1;
    const int pb = b ? gather_source_row(p, d, pair, s2) : -1;
    uint4 ra = make_uint4(0, 0, 0, 0), rb = ra;
    if (pa >= 0) ra = src[(size_t)pa * 16];
    if (pb >= 0) rb = src[(size_t)pb * 16];
    if (pa >= 0) dst0[(size_t)s * kSlotU4 + lane] = ra;
    if (pb >= 0) dst0[(size_t)s2 * kSlotU4 + lane] = rb;
  }
}

// ----------------------------------------------------------------------------- recompress
// Algorithm 2, the branch taken when the buffer is full: for every (sequence, semantic head) keep the top-M of the static
// set plus the buffered tokens by accumulated attention score (ties: lowest position) as the new
// static set; the buffer is then empty.  One CTA per pair.  Static tokens that stay keep their
// slots; the buffered tokens that make it take the slots of the static tokens that do not (and the
// still unused static slots), in ascending slot order.  So only the tokens that enter move (at most
// R rows per head, from the ring region into the static region: sources and destinations never
// overlap), and after the first re-selection the static slots are no longer ordered by position,
// which nothing depends on: ties are broken on the positions themselves.
__device__ __forceinline__ void recompress_pair(const RecompressParams& p, int pair) {
  extern __shared__ __align__(16) unsigned char rsm[];
  __shared__ uint32_t s_hist[256];
  __shared__ uint32_t s_prefix, s_need;
  __shared__ int s_nt, s_nsrc;
  const int seq = pair / p.H, head = pair - seq * p.H;
  const HeadDesc d = p.desc[head];
  if (!d.w) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int sv = p.static_valid;
  const int n = sv + p.buffered;                       // candidates: static slots, then buffer slots
  const int k = min(p.M, n);
  float* s_sc = reinterpret_cast<float*>(rsm);         // [mr] candidate scores
  int* s_pos = reinterpret_cast<int*>(s_sc + p.mr);    // [mr] candidate image indices
  int* s_flag = s_pos + p.mr;                          // [mr] 1 = kept
  int* s_tie = s_flag + p.mr;                          // [mr] candidates whose score equals the threshold
  int* s_src = s_tie + p.mr;                           // [mr] kept buffered candidates, buffer order
  int* s_dst = s_src + p.mr;                           // [mr] free static slots, ascending
  float* acc = p.acc + (size_t)pair * p.mr;
  int32_t* idx = p.static_idx + (size_t)pair * p.M;

  // candidate c lives in entry e(c) of the score row and of the head's static+ring slots
  for (int c = tid; c < n; c += kThreads) {
    const int e = c < sv ? c : d.y + (c - sv);
    float sc = acc[e];
    if (p.pending) {
      const float2 ml = p.ml[pair];
      sc += ex2(p.logits[(size_t)pair * p.mr + e] - ml.x) / ml.y;
    }
    s_sc[c] = sc;
    s_pos[c] = c < sv ? idx[c] : p.t_base + (c - sv);
  }
  if (tid == 0) { s_prefix = 0u; s_need = (uint32_t)k; s_nt = 0; s_nsrc = 0; }
  __syncthreads();

  const uint32_t* bits = reinterpret_cast<const uint32_t*>(s_sc);
  if (n <= kRankMax) {
    rank_select(bits, s_pos, n, k, s_flag);
  } else {
  // bit pattern of the k-th largest score (scores are non-negative)
  for (int shift = 24; shift >= 0; shift -= 8) {
    s_hist[tid] = 0u;
    __syncthreads();
    const uint32_t prefix = s_prefix;
    const uint32_t mask = shift == 24 ? 0u : (0xffffffffu << (shift + 8));
    for (int i0 = 0; i0 < n; i0 += kThreads) {
      const int i = i0 + tid;
      const uint32_t b = i < n ? bits[i] : 0u;
      hist_add(s_hist, i < n && (b & mask) == prefix, (b >> shift) & 255u);
    }
    __syncthreads();
    if (tid < 32) {
      uint32_t need = s_need;
      const int bin = pick_bin(s_hist, need, tid);
      if (tid == 0) {
        s_need = need;
        s_prefix = prefix | ((uint32_t)bin << shift);
      }
    }
    __syncthreads();
  }
  const uint32_t thr = s_prefix;
  const int need_eq = (int)s_need;

  // above the threshold: kept; equal to it: the need_eq lowest positions (positions are distinct)
  for (int c = tid; c < n; c += kThreads) {
    const uint32_t b = bits[c];
    s_flag[c] = b > thr ? 1 : 0;
    if (b == thr) s_tie[atomicAdd(&s_nt, 1)] = c;
  }
  __syncthreads();
  const int nt = s_nt;
  for (int i = tid; i < nt; i += kThreads) {
    const int c = s_tie[i], pc = s_pos[c];
    int rank = 0;
    for (int j = 0; j < nt; ++j) rank += s_pos[s_tie[j]] < pc ? 1 : 0;
    if (rank < need_eq) s_flag[c] = 1;
  }
  }
  __syncthreads();

  // who moves where: the j-th kept buffered token (buffer order) into the j-th free static slot
  // (slots of dropped static tokens and slots never used so far, ascending); one warp, by ballots
  if (warp == 0) {
    int cnt = 0;
    for (int c0 = sv; c0 < n; c0 += 32) {
      const int c = c0 + lane;
      const bool take = c < n && s_flag[c];
      const unsigned m = __ballot_sync(0xffffffffu, take);
      if (take) s_src[cnt + __popc(m & ((1u << lane) - 1u))] = c;
      cnt += __popc(m);
    }
    if (lane == 0) s_nsrc = cnt;
    cnt = 0;
    for (int o0 = 0; o0 < p.M; o0 += 32) {
      const int o = o0 + lane;
      const bool free_slot = o < p.M && (o >= sv || !s_flag[o]);
      const unsigned m = __ballot_sync(0xffffffffu, free_slot);
      if (free_slot) s_dst[cnt + __popc(m & ((1u << lane) - 1u))] = o;
      cnt += __popc(m);
    }
  }
  __syncthreads();
  const int nmove = s_nsrc;                            // free slots never run out: there are at least as many

  // scores and positions of the new static set
  for (int c = tid; c < sv; c += kThreads)
    if (s_flag[c]) acc[c] = s_sc[c];                   // with the last decode's weights folded in
  for (int j = tid; j < nmove; j += kThreads) {
    const int c = s_src[j], o = s_dst[j];
    acc[o] = s_sc[c];
    idx[o] = s_pos[c];
  }
  for (int o = k + tid; o < p.M; o += kThreads) idx[o] = -1;
  // rows of the tokens that enter: ring slot of buffer entry (c - sv) -> static slot
  uint4* hbase = p.slab + ((size_t)seq * p.seq_slots + d.x + p.L) * kSlotU4;
  for (int j = warp; j < nmove; j += kThreads / 32) {
    const int e = d.y + (s_src[j] - sv), o = s_dst[j];
    hbase[(size_t)o * kSlotU4 + lane] = hbase[(size_t)e * kSlotU4 + lane];
  }
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
  p.logits = q.logits + ((size_t)layer * 2 + ly.lg) * pairs * q.mr;
  p.ml = q.ml + ((size_t)layer * 2 + ly.lg) * pairs;
  p.pending = ly.pending;
  p.n_seqs = q.n_seqs; p.H = q.H; p.L = q.L; p.M = q.M; p.mr = q.mr;
  p.static_valid = ly.static_valid;
  p.buffered = ly.buffered;
  p.t_base = ly.t_base;
  p.seq_slots = ly.seq_slots;
  recompress_pair(p, blockIdx.x);
}

// Re-selection with a row buffer of ONE token (Algorithm 1 taken literally, one step): the token appended in
// the step just attended to either takes a still unused static slot, or the slot of the lowest-scoring static
// token (among equal scores the highest position leaves, so the new token loses ties), or is dropped itself.
// The same result as recompress_pair with one buffered token, without its rank counting and block-wide
// barriers: one warp per (layer, pair), which first adds the pending weights of the layer's last decode.
__global__ void __launch_bounds__(kThreads) ssd_evict_one_kernel(const __grid_constant__ RecompressLayersParams q) {
  const int lane = threadIdx.x & 31;
  const long long w = ((long long)blockIdx.x * kThreads + threadIdx.x) >> 5;
  const int pairs = q.n_seqs * q.H;
  if (w >= (long long)q.n_layers * pairs) return;
  const int layer = (int)(w / pairs), pair = (int)(w - (long long)layer * pairs);
  const RecompressLayer& ly = q.layer[layer];
  if (!ly.todo) return;
  const int seq = pair / q.H, head = pair - seq * q.H;
  const HeadDesc d = q.desc[(size_t)layer * q.H + head];
  if (!d.w) return;
  const size_t pr = (size_t)layer * pairs + pair;
  float* acc = q.acc + pr * q.mr;
  int32_t* idx = q.static_idx + pr * (q.M > 0 ? q.M : 1);
  const float* lg = q.logits + (((size_t)layer * 2 + ly.lg) * pairs + pair) * q.mr;
  float mx = 0.f, inv = 0.f;
  if (ly.pending) {
    const float2 ml = q.ml[((size_t)layer * 2 + ly.lg) * pairs + pair];
    mx = ml.x;
    inv = 1.f / ml.y;
  }
  const int sv = ly.static_valid;
  float worst = 3.0e38f;
  int worst_pos = -1, worst_e = -1;
  for (int i = lane; i < sv; i += 32) {
    float sc = acc[i];
    if (ly.pending) {
      sc += ex2(lg[i] - mx) * inv;
      acc[i] = sc;
    }
    const int pos = idx[i];
    if (sc < worst || (sc == worst && pos > worst_pos)) { worst = sc; worst_pos = pos; worst_e = i; }
  }
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) {
    const float w2 = __shfl_xor_sync(0xffffffffu, worst, off);
    const int p2 = __shfl_xor_sync(0xffffffffu, worst_pos, off), e2 = __shfl_xor_sync(0xffffffffu, worst_e, off);
    if (w2 < worst || (w2 == worst && p2 > worst_pos)) { worst = w2; worst_pos = p2; worst_e = e2; }
  }
  if (ly.buffered < 1) return;                       // nothing buffered: only the pending weights were due
  float w_new = acc[d.y];                            // entry of buffer slot 0
  if (ly.pending) w_new += ex2(lg[d.y] - mx) * inv;
  int dest = -1;
  if (sv < q.M) dest = sv;
  else if (sv > 0 && !(w_new <= worst)) dest = worst_e;
  __syncwarp();                                      // the scores written above, before the one written below
  if (dest < 0) return;
  if (lane == 0) {
    acc[dest] = w_new;
    idx[dest] = ly.t_base;
  }
  uint4* hb = q.slab + ((size_t)ly.first_slot + (size_t)seq * ly.seq_slots + d.x + q.L) * kSlotU4;
  hb[(size_t)dest * kSlotU4 + lane] = hb[(size_t)d.y * kSlotU4 + lane];
}

}  // namespace

cudaError_t launch_select(const SelectParams& p, cudaStream_t st) {
  ssd_select_kernel<<<p.n_seqs * p.H, kThreads, 0, st>>>(p);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_gather(const GatherParams& p, int max_slots, cudaStream_t st) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(p.n_seqs * p.H, (max_slots + 63) / 64 + 1);
  cfg.blockDim = dim3(kThreads);
  cfg.stream = st;
  // Only behind the selection kernel may the launch start early: behind anything else (the caller's kernel that
  // produced k_full, say) its first pass could read rows that are not written yet.
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = p.after_select ? 1 : 0;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, ssd_gather_kernel, p);
  count_launch();
  return e;
}

cudaError_t launch_recompress_layers(const RecompressLayersParams& p, cudaStream_t st) {
  if (p.n_layers < 1 || p.n_layers > kMaxLayersPerLaunch) return cudaErrorInvalidValue;
  const size_t smem = (size_t)(6 * p.mr + 4) * 4;
  cudaError_t e = cudaFuncSetAttribute(ssd_recompress_layers_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  ssd_recompress_layers_kernel<<<dim3(p.n_seqs * p.H, p.n_layers), kThreads, smem, st>>>(p);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_evict_one_layers(const RecompressLayersParams& p, cudaStream_t st) {
  if (p.n_layers < 1 || p.n_layers > kMaxLayersPerLaunch) return cudaErrorInvalidValue;
  const long long warps = (long long)p.n_layers * p.n_seqs * p.H;
  ssd_evict_one_kernel<<<(unsigned)((warps * 32 + kThreads - 1) / kThreads), kThreads, 0, st>>>(p);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_recompress(const RecompressParams& p, cudaStream_t st) {
  const size_t smem = (size_t)(6 * p.mr + 4) * 4;
  cudaError_t e = cudaFuncSetAttribute(ssd_recompress_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  ssd_recompress_kernel<<<p.n_seqs * p.H, kThreads, smem, st>>>(p);
  count_launch();
  return cudaGetLastError();
}

}  // namespace ssd
