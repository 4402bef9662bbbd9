// The dense contraction of the method on the 5th-generation tensor cores: logit tiles
//   S[128 query rows, 128 keys] = Q_tile K_tile^T   (bf16 x bf16 -> fp32, head dimension 128)
// computed by tcgen05.mma with both operands in shared memory and the accumulator in tensor
// memory (TMEM), and consumed in place: every thread owns one query row (one TMEM lane) and reads
// its 128 logits with tcgen05.ld, so the softmax statistics of a row need no cross-thread step.
//
// Used by the head classifier (Sec. 3.3 sparsity metric): per image step t, the attention mass on
// visual tokens older than the newest w, over the mass on all visual tokens so far.  Only visual
// columns are touched: the prompt's share of the softmax cancels in the ratio.
// Used by the sink scoring of ssd_compress (Algorithm 1, AttentionScores and running sum): per
// block of 128 observed queries, a first sweep over the key tiles gives every row its maximum and
// exp-sum, a second sweep recomputes the tiles, normalises, and adds the columns up.  The sum over
// the 32 rows of a warp is a shuffle transpose-reduction; each warp keeps its own score array in
// shared memory and the four are added in a fixed order at the end, so scores are bitwise
// reproducible from run to run, which the selection relies on.
//
// Operand tiles sit in shared memory in the K-major layout without swizzling: 8 rows x 16 bytes
// form a contiguous 128-byte core matrix, core matrices follow each other along the head
// dimension (128 bytes apart) and groups of 8 rows follow each other 2048 bytes apart.  Tiles are
// written with 16-byte cp.async (zero fill past the end of the tensor).  One CTA = one block of
// 128 query rows of one (layer, sequence, head); several CTAs per SM overlap each other's loads,
// MMAs and exponentials.  Every mbarrier wait is bounded and failures end in the status word.
#include "ssd_internal.cuh"

namespace ssd {

namespace {

constexpr int kRows = 128;                 // query rows per CTA = TMEM lanes = threads
constexpr int kKeys = 128;                 // keys per tile = TMEM columns of one accumulator
constexpr int kTileBytes = 128 * kHeadDim * 2;   // 32 KB per operand tile
constexpr int kLbo = 128;                  // bytes between core matrices along the head dimension
constexpr int kSbo = 2048;                 // bytes between groups of 8 rows
constexpr float kNegBig = -1.0e30f;
constexpr unsigned long long kWaitLimitNs = 1000000000ull;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// ---- mbarrier with a bounded wait
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  bool ok = mbar_try_wait(bar, parity);
  if (!ok) {
    const unsigned long long t0 = global_ns();
    do {
#pragma unroll 1
      for (int i = 0; i < 64 && !ok; ++i) ok = mbar_try_wait(bar, parity);
    } while (!ok && global_ns() - t0 < kWaitLimitNs);
  }
  return ok;
}

// ---- operand tiles
// Copy rows [row0, row0 + 128) of a row-major [n_rows, 128] bf16 matrix into a tile (zero rows past
// n_rows).  A warp moves 8 rows x 64 bytes per step: full 32-byte sectors on the global side,
// conflict-free 128-byte runs on the shared side.
__device__ __forceinline__ void load_tile(uint32_t tile_s, const __nv_bfloat16* __restrict__ src, int row0, int n_rows,
                                          int warp, int lane, int n_warps) {
  const int r8 = lane & 7, c4 = lane >> 3;
  for (int it = warp; it < 16 * 4; it += n_warps) {
    const int rg = it >> 2, cg = it & 3;          // group of 8 rows, group of 4 chunks
    const int r = rg * 8 + r8, c = cg * 4 + c4;   // row in tile, 16-byte chunk in row
    const int grow = row0 + r;
    const bool in = grow < n_rows;
    const __nv_bfloat16* g = src + (size_t)(in ? grow : 0) * kHeadDim + c * 8;
    const uint32_t dst = tile_s + (uint32_t)(rg * kSbo + c * kLbo + r8 * 16);
    const int bytes = in ? 16 : 0;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(g), "r"(bytes) : "memory");
  }
}
__device__ __forceinline__ void tiles_ready_for_mma() {
  asm volatile("cp.async.wait_all;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes -> tensor-core reads
}

// Shared-memory matrix descriptor of a K-major, unswizzled operand starting at byte address `addr`.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
  const uint32_t lo = ((addr >> 4) & 0x3fffu) | ((uint32_t)(kLbo >> 4) << 16);
  const uint32_t hi = (uint32_t)(kSbo >> 4) | (1u << 14);        // descriptor version 1, no swizzle
  return ((uint64_t)hi << 32) | lo;
}
// Instruction descriptor: D = fp32, A = B = bf16, both K-major, N = 128, M = 128.
constexpr uint32_t kInstrDesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kKeys >> 3) << 17) |
                                ((uint32_t)(kRows >> 4) << 24);

// One thread: S[128 x 128] (TMEM columns [tmem_d, tmem_d + 128)) = A_tile B_tile^T, then signal `bar`.
__device__ __forceinline__ void mma_tile(uint32_t tmem_d, uint32_t a_s, uint32_t b_s, uint32_t bar) {
#pragma unroll
  for (int k = 0; k < kHeadDim / 16; ++k) {
    const uint64_t da = smem_desc(a_s + k * 2 * kLbo), db = smem_desc(b_s + k * 2 * kLbo);
    const uint32_t accumulate = k > 0 ? 1u : 0u;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n" ::"r"(tmem_d), "l"(da), "l"(db), "r"(kInstrDesc), "r"(accumulate)
        : "memory");
  }
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// 32 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
}

// Running softmax statistics of one row over the visual keys: exp-sum over all visible keys and over
// the "far" ones (older than the newest w), both relative to the running maximum m (base-2 units).
struct RowStats {
  float m, all, far;
};

// Fold 32 logits (raw dot products; x = v * scale) of keys base .. base + 31 into the statistics of
// the row whose newest visible key is `row` and whose newest far key is `row - w`.
__device__ __forceinline__ void fold32(RowStats& st, const float (&v)[32], int base, int row, int w, float scale) {
  const int nv = min(max(row - base + 1, 0), 32);          // visible: first nv
  const int nf = min(max(row - w - base + 1, 0), 32);      // far: first nf
  if (nv == 0) return;
  float gmax = kNegBig;
#pragma unroll
  for (int j = 0; j < 32; ++j) gmax = fmaxf(gmax, j < nv ? v[j] : kNegBig);
  const float mn = fmaxf(st.m, gmax * scale);
  const float corr = ex2(st.m - mn);
  float sa = 0.f, sf = 0.f;
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    const float e = j < nv ? ex2(fmaf(v[j], scale, -mn)) : 0.f;
    sa += e;
    sf += j < nf ? e : 0.f;
  }
  st.all = st.all * corr + sa;
  st.far = st.far * corr + sf;
  st.m = mn;
}

// ----------------------------------------------------------------------------- classify
// One CTA per (unit, block of 128 image steps), unit = (layer, calibration sequence, head).
__global__ void __launch_bounds__(kRows) ssd_classify_kernel(const ClassifyParams p, int n_row_blocks) {
  extern __shared__ __align__(1024) unsigned char smem[];
  __shared__ uint64_t s_bar;
  __shared__ uint32_t s_tmem;
  __shared__ float s_ratio[4];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int unit = blockIdx.x / n_row_blocks, rb = blockIdx.x - unit * n_row_blocks;
  const __nv_bfloat16* Q = p.q_cal + (size_t)unit * p.N * kHeadDim;
  const __nv_bfloat16* K = p.k_cal + ((size_t)unit * (p.L + p.N) + p.L) * kHeadDim;   // visual keys
  const int r0 = rb * kRows;
  const int row = r0 + tid;                 // image index of this thread's query; step t = row + 1
  const int last_row = min(r0 + kRows, p.N) - 1;

  const uint32_t q_s = smem_u32(smem), k_s = q_s + kTileBytes;
  const uint32_t bar = smem_u32(&s_bar);
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)), "r"(kKeys)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (tid == 0) {
    mbar_init(bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  load_tile(q_s, Q, r0, p.N, warp, lane, 4);
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = s_tmem;
  const uint32_t my_tmem = tmem + ((uint32_t)(warp * 32) << 16);

  RowStats st = {kNegBig, 0.f, 0.f};
  uint32_t parity = 0;
  bool ok = true;
  for (int k0 = 0; k0 <= last_row; k0 += kKeys) {
    load_tile(k_s, K, k0, p.N, warp, lane, 4);
    tiles_ready_for_mma();
    __syncthreads();
    if (tid == 0) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      mma_tile(tmem, q_s, k_s, bar);
    }
    ok = mbar_wait(bar, parity);
    parity ^= 1u;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (__all_sync(0xffffffffu, ok)) {
      const int warp_last = min(r0 + warp * 32 + 31, last_row);
#pragma unroll 1
      for (int cb = 0; cb < kKeys / 32; ++cb) {
        const int base = k0 + cb * 32;
        if (base > warp_last) break;          // no row of this warp sees these keys
        float v[32];
        tmem_ld32(my_tmem + cb * 32, v);
        if (row < p.N) fold32(st, v, base, row, p.w, p.scale_log2);
      }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    // everyone is done with the key tile and the accumulator; a CTA-wide verdict on the wait
    if (!__syncthreads_and(ok ? 1 : 0)) {
      ok = false;
      break;
    }
  }

  float ratio = (ok && row < p.N && st.all > 0.f) ? st.far / st.all : 0.f;
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) ratio += __shfl_xor_sync(0xffffffffu, ratio, o);
  if (lane == 0) s_ratio[warp] = ratio;
  __syncthreads();
  if (tid == 0) {
    p.ratio_part[(size_t)unit * n_row_blocks + rb] = (s_ratio[0] + s_ratio[1]) + (s_ratio[2] + s_ratio[3]);
    if (!ok) atomicOr(p.status, 2u);
  }
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kKeys) : "memory");
  }
}

// ----------------------------------------------------------------------------- score
// Sum over the 32 lanes of a warp of 32 values each: lane j returns the total of value j.
__device__ __forceinline__ float warp_column_sums(float (&a)[32], int lane) {
#pragma unroll
  for (int s = 16; s >= 1; s >>= 1) {
    const bool up = (lane & s) != 0;
#pragma unroll
    for (int i = 0; i < s; ++i) {
      const float keep = up ? a[i + s] : a[i];
      const float send = up ? a[i] : a[i + s];
      a[i] = keep + __shfl_xor_sync(0xffffffffu, send, s);
    }
  }
  return a[0];
}

// One CTA per (sequence, semantic head); loops over blocks of 128 observed queries.
__global__ void __launch_bounds__(kRows) ssd_score_kernel(const ScoreParams p) {
  extern __shared__ __align__(1024) unsigned char smem[];
  __shared__ uint64_t s_bar;
  __shared__ uint32_t s_tmem;
  const int pair = blockIdx.x;
  const int head = pair % p.H;
  if (!p.desc[head].w) return;            // before any tensor-memory allocation
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int ctx_all = p.L + p.n0;
  const __nv_bfloat16* Q = p.q_obs + (size_t)pair * p.n_obs * kHeadDim;
  const __nv_bfloat16* K = p.k_full + (size_t)pair * ctx_all * kHeadDim;
  const int t_first = p.n0 - p.n_obs + 1;  // image step of observed row 0

  const uint32_t q_s = smem_u32(smem), k_s = q_s + kTileBytes;
  float* s_score = reinterpret_cast<float*>(smem + 2 * kTileBytes);   // [4 warps][n0]
  const uint32_t bar = smem_u32(&s_bar);
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)), "r"(kKeys)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (tid == 0) {
    mbar_init(bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int j = tid; j < 4 * p.n0; j += kRows) s_score[j] = 0.f;
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = s_tmem;
  const uint32_t my_tmem = tmem + ((uint32_t)(warp * 32) << 16);
  float* my_score = s_score + (size_t)warp * p.n0;

  uint32_t parity = 0;
  bool ok = true;
  // S tile of keys [k0, k0 + 128) for the current query block; false if the wait ran out
  auto logits_tile = [&](int k0) -> bool {
    load_tile(k_s, K, k0, ctx_all, warp, lane, 4);
    tiles_ready_for_mma();
    __syncthreads();
    if (tid == 0) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      mma_tile(tmem, q_s, k_s, bar);
    }
    const bool done = mbar_wait(bar, parity);
    parity ^= 1u;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    return __all_sync(0xffffffffu, done);
  };
  // everyone is done with the key tile and the accumulator; a CTA-wide verdict on the wait
  auto tile_done = [&](bool fine) -> bool {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    return __syncthreads_and(fine ? 1 : 0) != 0;
  };

  for (int r0 = 0; r0 < p.n_obs && ok; r0 += kRows) {
    load_tile(q_s, Q, r0, p.n_obs, warp, lane, 4);
    const int row = r0 + tid;
    const int ctx_r = row < p.n_obs ? p.L + t_first + row : 0;        // keys [0, ctx_r) are visible
    const int last = min(r0 + kRows, p.n_obs) - 1;
    const int ctx_max = p.L + t_first + last;                        // context of the block's last row
    const int warp_ctx = p.L + t_first + min(r0 + warp * 32 + 31, last);

    // sweep 1: row maximum and exp-sum
    RowStats st = {kNegBig, 0.f, 0.f};
    for (int k0 = 0; k0 < ctx_max && ok; k0 += kKeys) {
      const bool fine = logits_tile(k0);
      if (fine) {
#pragma unroll 1
        for (int cb = 0; cb < kKeys / 32; ++cb) {
          const int base = k0 + cb * 32;
          if (base >= warp_ctx) break;
          float v[32];
          tmem_ld32(my_tmem + cb * 32, v);
          fold32(st, v, base, ctx_r - 1, 0, p.scale_log2);
        }
      }
      ok = tile_done(fine);
    }
    const float inv = st.all > 0.f ? 1.f / st.all : 0.f;

    // sweep 2: normalised probabilities, column sums over the block's rows
    for (int k0 = (p.L / kKeys) * kKeys; k0 < ctx_max && ok; k0 += kKeys) {
      const bool fine = logits_tile(k0);
      if (fine) {
#pragma unroll 1
        for (int cb = 0; cb < kKeys / 32; ++cb) {
          const int base = k0 + cb * 32;
          if (base >= warp_ctx) break;
          if (base + 32 <= p.L) continue;                 // prompt keys only: not scored
          float v[32];
          tmem_ld32(my_tmem + cb * 32, v);
          const int nv = min(max(ctx_r - base, 0), 32);
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = j < nv ? ex2(fmaf(v[j], p.scale_log2, -st.m)) * inv : 0.f;
          const float col = warp_column_sums(v, lane);
          const int key = base + lane;
          if (key >= p.L && key < ctx_max) my_score[key - p.L] += col;
        }
      }
      ok = tile_done(fine);
    }
  }

  __syncthreads();
  float* out = p.score + (size_t)pair * p.n0;
  for (int j = tid; j < p.n0; j += kRows)
    out[j] = ok ? (s_score[j] + s_score[p.n0 + j]) + (s_score[2 * p.n0 + j] + s_score[3 * p.n0 + j]) : 0.f;
  if (tid == 0 && !ok) atomicOr(p.status, 4u);
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kKeys) : "memory");
  }
}

}  // namespace

int classify_rows_per_block() { return kRows; }

cudaError_t launch_classify(const ClassifyParams& p, int n_row_blocks, cudaStream_t st) {
  const int smem = 2 * kTileBytes + 1024;
  cudaError_t e = cudaFuncSetAttribute(ssd_classify_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  ssd_classify_kernel<<<p.n_units * n_row_blocks, kRows, smem, st>>>(p, n_row_blocks);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_score(const ScoreParams& p, cudaStream_t st) {
  const size_t smem = 2 * (size_t)kTileBytes + 4 * (size_t)p.n0 * sizeof(float) + 1024;
  if (smem > 227 * 1024) return cudaErrorInvalidValue;
  cudaError_t e = cudaFuncSetAttribute(ssd_score_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  ssd_score_kernel<<<p.n_seqs * p.H, kRows, smem, st>>>(p);
  count_launch();
  return cudaGetLastError();
}

}  // namespace ssd
