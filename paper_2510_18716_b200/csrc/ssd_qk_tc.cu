// The dense contraction of the method on the 5th-generation tensor cores: logit tiles
//   S[128 query rows, 128 keys] = Q_tile K_tile^T   (bf16 x bf16 -> fp32, head dimension 128)
// computed by tcgen05.mma with both operands in shared memory and the accumulator in tensor
// memory (TMEM), and consumed in place with tcgen05.ld.
//
// Used by the head classifier (Sec. 3.3 sparsity metric): per image step t, the attention mass on
// visual tokens older than the newest w, over the mass on all visual tokens so far.  Only visual
// columns are touched: the prompt's share of the softmax cancels in the ratio.
// Used by the sink scoring of ssd_compress (Algorithm 1, AttentionScores and running sum): per
// block of 128 observed queries, a first sweep over the key tiles gives every row its maximum and
// exp-sum; a second sweep recomputes the tiles TRANSPOSED (S^T = K_tile Q_tile^T: the operands swap
// roles, the shared-memory tiles are the same), so that a TMEM lane is a key and a thread adds up its
// key's normalised probabilities over the queries in its own registers: no exchange between lanes.
// What a query's logits are normalised by, m + log2(exp-sum), then differs from column to column of a
// thread's accumulator row; it is subtracted by the tensor core: one more MMA step per tile adds the
// rank-one term 1 (a_1 + a_2 + a_3)^T, where a_1 + a_2 + a_3 is the three-term bf16 expansion of
// -(m + log2 l) / scale of each query (exact to 2^-24), from two small operand tiles that the epilogue
// warps write (no-swizzle K-major layout), so the exponent is one multiplication away from the accumulator.
// The two warps that share a lane quadrant take one half of the queries each and keep a score row
// each in global memory (it stays in L2; every element belongs to one lane of one warp, which adds
// to it with reductions that return nothing), and the selection adds the rows in a fixed order, so
// scores are bitwise reproducible from run to run, which it relies on.
//
// A CTA is a pipeline of three roles that meet only at mbarriers:
//   warp 0, one lane   producer: TMA (cp.async.bulk.tensor, 128-byte swizzle) brings the query tile
//                      of a row block and the key tiles, the latter into a ring of kStages buffers;
//   warp 1, one lane   issues the 8 tcgen05.mma of a tile into one of kAccs TMEM accumulators and
//                      commits them to the barriers that free the key stage and publish the tile;
//   warps 2..9         read the accumulator (tcgen05.ld), hand it back as soon as it is in registers
//                      and do the exponentials.  A query row (one TMEM lane) belongs to two threads,
//                      one per half of the tile's columns; the halves of a row's softmax statistics
//                      meet through shared memory.
// so the loads and the MMAs of tile k+1 run under the exponentials of tile k.  Two CTAs share an SM
// (2 x 96 KB of tiles, 2 x 256 TMEM columns).  Operand tiles are two TMA boxes of 128 rows x 64
// elements in the K-major 128-byte-swizzled layout (8-row groups 1024 bytes apart); rows past the
// end of a tensor are zero-filled by the TMA unit.  Every mbarrier wait is bounded: a wait that
// runs out raises the CTA's abort flag, after which no role waits any more, all of them run to the
// end of their loops, the CTA reports through the status word and frees its tensor memory.
#include <cuda.h>

#include "ssd_internal.cuh"
#include "ssd_device.cuh"

namespace ssd {

namespace {

constexpr int kRows = 128;                 // query rows per block = TMEM lanes
constexpr int kKeys = 128;                 // keys per tile = TMEM columns of one accumulator
constexpr int kBoxBytes = 128 * 64 * 2;    // one TMA box: 128 rows x 64 bf16
constexpr int kTileBytes = 2 * kBoxBytes;  // 32 KB per operand tile (two boxes along the head dimension)
constexpr int kStages = 2;                 // key tiles in flight
constexpr int kAccs = 2;                   // TMEM accumulators
constexpr int kEpiWarps = 8;
constexpr int kEpiThreads = kEpiWarps * 32;
constexpr int kTcThreads = 64 + kEpiThreads;
constexpr int kTmemCols = kAccs * kKeys;   // 256: a power of two, as the allocator wants
static_assert(kHeadDim == 128, "two 64-element boxes per tile row");

// ---- every wait on an mbarrier is bounded and gives up at once when the CTA's abort flag is up
__device__ __forceinline__ bool pipe_wait(uint32_t bar, uint32_t parity, volatile int* abort) {
  if (*abort) return false;
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (*abort) return false;
    if (global_ns() - t0 > kWaitLimitNs) {
      *abort = 1;
      return false;
    }
  }
}

// The barriers of a CTA's pipeline, one after another in shared memory; `base` is the address of the first.
struct PipeBars {
  uint64_t b[2 + 2 * kStages + 2 * kAccs + 1];
};
struct Pipe {
  uint32_t base;
  __device__ __forceinline__ uint32_t q_full() const { return base; }
  __device__ __forceinline__ uint32_t q_empty() const { return base + 8; }
  __device__ __forceinline__ uint32_t full(int s) const { return base + 16 + 8 * s; }
  __device__ __forceinline__ uint32_t empty(int s) const { return base + 16 + 8 * (kStages + s); }
  __device__ __forceinline__ uint32_t acc_full(int a) const { return base + 16 + 8 * (2 * kStages + a); }
  __device__ __forceinline__ uint32_t acc_empty(int a) const { return base + 16 + 8 * (2 * kStages + kAccs + a); }
  // scoring only: the normalisers of a query block are in their operand tile (one arrival per writing warp)
  __device__ __forceinline__ uint32_t ext_full() const { return base + 16 + 8 * (2 * kStages + 2 * kAccs); }
};
__device__ __forceinline__ Pipe pipe_make(PipeBars& bars, bool init) {
  Pipe p;
  p.base = smem_u32(&bars.b[0]);
  if (init) {
    mbar_init(p.q_full(), 1);
    mbar_init(p.q_empty(), 1);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(p.full(s), 1);
      mbar_init(p.empty(s), 1);
    }
    for (int a = 0; a < kAccs; ++a) {
      mbar_init(p.acc_full(a), 1);
      mbar_init(p.acc_empty(a), kEpiWarps);
    }
    mbar_init(p.ext_full(), kEpiWarps / 2);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  return p;
}

// ---- operand tiles
// Bring a tensor map (a kernel parameter) towards the TMA unit before its first use.
__device__ __forceinline__ void prefetch_map(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}
// One box of a tile: rows [y, y + 128) x elements [x, x + 64) of unit z of a [units, rows, 128] bf16
// tensor.  x is 0 or 64 (128 bytes), so the copy starts on the boundary the TMA unit wants.
__device__ __forceinline__ void tma_box(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tma_tile(uint32_t dst, const CUtensorMap* map, int row0, int unit, uint32_t bar) {
  mbar_expect_tx(bar, kTileBytes);
  tma_box(dst, map, 0, row0, unit, bar);
  tma_box(dst + kBoxBytes, map, 64, row0, unit, bar);
}

// Shared-memory matrix descriptor of a K-major operand in the 128-byte-swizzled layout starting at
// byte address `addr`: groups of 8 rows 1024 bytes apart, descriptor version 1.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
  const uint32_t lo = ((addr >> 4) & 0x3fffu) | (1u << 16);
  const uint32_t hi = (uint32_t)(1024 >> 4) | (1u << 14) | (2u << 29);
  return ((uint64_t)hi << 32) | lo;
}
// Instruction descriptor: D = fp32, A = B = bf16, both K-major, N = 128, M = 128.
constexpr uint32_t kInstrDesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kKeys >> 3) << 17) |
                                ((uint32_t)(kRows >> 4) << 24);

// One thread: S[128 x 128] (TMEM columns [tmem_d, tmem_d + 128)) = A_tile B_tile^T.  A step of 16
// elements along the head dimension is 32 bytes inside a swizzled row; the second box follows the first.
__device__ __forceinline__ void mma_tile(uint32_t tmem_d, uint32_t a_s, uint32_t b_s) {
#pragma unroll
  for (int k = 0; k < kHeadDim / 16; ++k) {
    const uint32_t off = (uint32_t)((k >> 2) * kBoxBytes + (k & 3) * 32);
    const uint64_t da = smem_desc(a_s + off), db = smem_desc(b_s + off);
    const uint32_t accumulate = k > 0 ? 1u : 0u;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n" ::"r"(tmem_d), "l"(da), "l"(db), "r"(kInstrDesc), "r"(accumulate)
        : "memory");
  }
}
// A 128 x 16 bf16 operand without swizzle, K-major, in the canonical layout of 8-row x 16-byte core matrices:
// [group of 8 rows][half of the 16 elements][row in group][16 bytes], i.e. 256 bytes from one group of rows to
// the next and 128 bytes between the two core matrices of a group along K.
constexpr int kExtTileBytes = 128 * 16 * 2;
constexpr int kExtBytes = 2 * kExtTileBytes;     // the tile of ones, then the tile of normalisers
__device__ __forceinline__ uint64_t smem_desc_plain(uint32_t addr) {
  const uint32_t lo = ((addr >> 4) & 0x3fffu) | ((uint32_t)(128 >> 4) << 16);
  const uint32_t hi = (uint32_t)(256 >> 4) | (1u << 14);
  return ((uint64_t)hi << 32) | lo;
}
__device__ __forceinline__ uint32_t ext_row_offset(int row) { return (uint32_t)((row >> 3) * 256 + (row & 7) * 16); }
// One thread: S[128 x 128] += A_ext B_ext^T, one step of 16 along K.
__device__ __forceinline__ void mma_ext(uint32_t tmem_d, uint32_t a_s, uint32_t b_s) {
  const uint64_t da = smem_desc_plain(a_s), db = smem_desc_plain(b_s);
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
      "}\n" ::"r"(tmem_d), "l"(da), "l"(db), "r"(kInstrDesc), "r"(1u)
      : "memory");
}
// The barrier gets one arrival when every tcgen05.mma this thread has issued so far is complete.
__device__ __forceinline__ void mma_commit(uint32_t bar) {
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

// ---- the three roles.  Each keeps its own count of tiles (t) and query blocks (qn); stage, accumulator
// and barrier phase follow from the counts, so the roles agree as long as they walk the same schedule.
struct Producer {
  Pipe p;
  volatile int* abort;
  uint32_t q_s, k_s;
  const CUtensorMap *tq, *tk;
  int t = 0, qn = 0;
  int q_last = -1, k_last = -1;       // counts of the last copies actually issued (-1: none)
  __device__ __forceinline__ void query_block(int row0, int unit) {
    pipe_wait(p.q_empty(), ((qn & 1) ^ 1), abort);        // the MMAs of the previous block are done with it
    if (!*abort) {
      tma_tile(q_s, tq, row0, unit, p.q_full());
      q_last = qn;
    }
    ++qn;
  }
  __device__ __forceinline__ void key_tile(int row0, int unit) {
    const int s = t % kStages;
    pipe_wait(p.empty(s), ((t / kStages) & 1) ^ 1, abort);
    if (!*abort) {
      tma_tile(k_s + s * kTileBytes, tk, row0, unit, p.full(s));
      k_last = t;
    }
    ++t;
  }
  // After an abort: give the copies still in flight their time to land before the CTA ends.
  __device__ __forceinline__ void drain() {
    if (!*abort) return;
    const unsigned long long t0 = global_ns();
    bool done = false;
    while (!done && global_ns() - t0 < kWaitLimitNs) {
      done = q_last < 0 || mbar_try_wait(p.q_full(), q_last & 1);
      for (int d = 0; d < kStages; ++d) {
        const int tt = k_last - d;     // the stages hold the last kStages tiles issued
        if (tt >= 0) done = mbar_try_wait(p.full(tt % kStages), (tt / kStages) & 1) && done;
      }
    }
  }
};

struct Issuer {
  Pipe p;
  volatile int* abort;
  uint32_t q_s, k_s, tmem;
  uint32_t ext_s = 0;          // scoring: the tile of ones, then the tile of normalisers
  int t = 0, qn = 0;
  __device__ __forceinline__ void query_block() { pipe_wait(p.q_full(), qn & 1, abort); }
  // scoring: the block's normalisers are written (and visible to the tensor core)
  __device__ __forceinline__ void normalisers() {
    pipe_wait(p.ext_full(), qn & 1, abort);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  }
  // transposed: the accumulator gets S^T (lanes = keys, columns = queries) instead of S, minus every query's
  // normaliser.  first: the block's first such tile; its eight steps over the head dimension do not need the
  // normalisers and are issued before the wait for them, so the tensor core works while the epilogue warps finish
  // the first sweep.
  __device__ __forceinline__ void key_tile(bool transposed = false, bool first = false) {
    const int s = t % kStages, a = t % kAccs;
    pipe_wait(p.full(s), (t / kStages) & 1, abort);
    pipe_wait(p.acc_empty(a), ((t / kAccs) & 1) ^ 1, abort);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (!*abort) {
      if (transposed) mma_tile(tmem + a * kKeys, k_s + s * kTileBytes, q_s);
      else mma_tile(tmem + a * kKeys, q_s, k_s + s * kTileBytes);
    }
    if (first) normalisers();
    if (!*abort) {
      if (transposed) mma_ext(tmem + a * kKeys, ext_s, ext_s + kExtTileBytes);
      mma_commit(p.empty(s));
      mma_commit(p.acc_full(a));
    }
    ++t;
  }
  __device__ __forceinline__ void end_block() {
    if (!*abort) mma_commit(p.q_empty());
    ++qn;
  }
};

struct Consumer {
  Pipe p;
  volatile int* abort;
  uint32_t tmem_lane;        // TMEM address of this warp's lane quadrant, column 0
  int lane;
  int t = 0;
  // waits for the tile; returns the TMEM address of this warp's lanes of its accumulator
  __device__ __forceinline__ uint32_t tile() {
    const int a = t % kAccs;
    pipe_wait(p.acc_full(a), (t / kAccs) & 1, abort);
    __syncwarp();              // the lanes left the wait one by one; tcgen05.ld wants them together
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    return tmem_lane + a * kKeys;
  }
  // this warp has read all it wants from the tile's accumulator
  __device__ __forceinline__ void release() {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncwarp();
    if (lane == 0) mbar_arrive(p.acc_empty(t % kAccs));
    ++t;
  }
};

// ---- softmax statistics
// Running statistics of one row over its column half: exp-sum over all visible keys and over the
// "far" ones (older than the newest w), both relative to the running maximum m (base-2 units).
struct RowStats {
  float m, all, far;
};

// Fold 32 logits (raw dot products; x = v * scale) into the statistics of a row that sees the first
// nv of them, the first nf of which are far.  Without kMasked the row sees all 32 and they are
// either all far or none (all_far); without kFar the far sum is not kept.
template <bool kMasked, bool kFar>
__device__ __forceinline__ void fold32(RowStats& st, const float (&v)[32], int nv, int nf, bool all_far, float scale) {
  if (kMasked && nv <= 0) return;
  float gmax = kNegBig;
#pragma unroll
  for (int j = 0; j < 32; ++j) gmax = fmaxf(gmax, (!kMasked || j < nv) ? v[j] : kNegBig);
  const float mn = fmaxf(st.m, gmax * scale);
  const float corr = ex2(st.m - mn);
  float sa = 0.f, sf = 0.f;
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    const float e = (!kMasked || j < nv) ? ex2(fmaf(v[j], scale, -mn)) : 0.f;
    sa += e;
    if (kMasked && kFar) sf += j < nf ? e : 0.f;
  }
  if (!kMasked && kFar) sf = all_far ? sa : 0.f;
  st.all = st.all * corr + sa;
  if (kFar) st.far = st.far * corr + sf;
  st.m = mn;
}

__device__ __forceinline__ int clamp32(int x) { return min(max(x, 0), 32); }

// What every CTA does first: barriers, abort flag, tensor memory.  Returns the 1024-byte aligned
// shared-memory address of the tiles (query tile, then the key stages).
__device__ __forceinline__ uint32_t cta_setup(unsigned char* smem, PipeBars& bars, uint32_t* s_tmem, int* s_abort, Pipe& pipe) {
  const int tid = threadIdx.x, warp = tid >> 5;
  if (tid == 0) *s_abort = 0;
  pipe = pipe_make(bars, tid == 0);
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  return (smem_u32(smem) + 1023u) & ~1023u;
}
__device__ __forceinline__ void cta_teardown(uint32_t tmem) {
  if (threadIdx.x < 32) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

// ----------------------------------------------------------------------------- classify
// One CTA = one block of 128 query rows of one unit (layer, calibration sequence, head); its key
// tiles are those up to the diagonal.  Blocks of a unit are launched longest first.
__global__ void __launch_bounds__(kTcThreads, 2)
ssd_classify_kernel(const ClassifyParams p, int n_row_blocks, const __grid_constant__ CUtensorMap tq,
                    const __grid_constant__ CUtensorMap tk) {
  extern __shared__ __align__(1024) unsigned char smem[];
  __shared__ PipeBars s_bars;
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort;
  __shared__ float s_ratio[4];
  __shared__ float s_half[3][kRows];        // statistics of the rows' upper column halves
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int unit = blockIdx.x / n_row_blocks;
  const int rb = n_row_blocks - 1 - (blockIdx.x - unit * n_row_blocks);
  const int r0 = rb * kRows;
  const int last_row = min(r0 + kRows, p.N) - 1;
  const int n_tiles = last_row / kKeys + 1;   // keys 0 .. last_row

  if (tid == 0) {                      // while the thread block sets itself up
    prefetch_map(&tq);
    prefetch_map(&tk);
  }
  Pipe pipe;
  const uint32_t q_s = cta_setup(smem, s_bars, &s_tmem, &s_abort, pipe), k_s = q_s + kTileBytes;
  const uint32_t tmem = s_tmem;

  const int quad = warp & 3, half = (warp - 2) >> 2;   // TMEM lane quadrant; which half of a tile's columns
  const int rl = quad * 32 + lane;                     // row inside the block
  const int row = r0 + rl;                             // image index of this thread's query; step t = row + 1
  RowStats st = {kNegBig, 0.f, 0.f};

  if (warp == 0) {
    if (lane == 0) {
      Producer pr;
      pr.p = pipe; pr.abort = &s_abort; pr.q_s = q_s; pr.k_s = k_s; pr.tq = &tq; pr.tk = &tk;
      pr.query_block(r0, unit);
      for (int ti = 0; ti < n_tiles; ++ti) pr.key_tile(p.L + ti * kKeys, unit);   // visual keys only
      pr.drain();
    }
  } else if (warp == 1) {
    if (lane == 0) {
      Issuer is;
      is.p = pipe; is.abort = &s_abort; is.q_s = q_s; is.k_s = k_s; is.tmem = tmem;
      is.query_block();
      for (int ti = 0; ti < n_tiles; ++ti) is.key_tile();
      is.end_block();
    }
  } else {
    Consumer co;
    co.p = pipe; co.abort = &s_abort; co.tmem_lane = tmem + ((uint32_t)(quad * 32) << 16); co.lane = lane;
    const int lo_row = r0 + quad * 32;                  // this warp's rows: lo_row .. lo_row + 31
    const int warp_last = min(lo_row + 31, last_row);
    for (int ti = 0; ti < n_tiles; ++ti) {
      const uint32_t acc = co.tile();
      bool released = false;
#pragma unroll 1
      for (int cb = 2 * half; cb < 2 * half + 2; ++cb) {
        const int base = ti * kKeys + cb * 32;
        if (base > warp_last || lo_row > last_row) break;   // no row of this warp sees these keys
        float v[32];
        tmem_ld32(acc + cb * 32, v);
        if (cb == 2 * half + 1) {
          co.release();
          released = true;
        }
        const bool all_far = base + 31 <= lo_row - p.w, none_far = base > lo_row + 31 - p.w;
        if (base + 31 <= lo_row && (all_far || none_far)) {
          fold32<false, true>(st, v, 32, 0, all_far, p.scale_log2);
        } else if (row < p.N) {
          fold32<true, true>(st, v, clamp32(row - base + 1), clamp32(row - p.w - base + 1), false, p.scale_log2);
        }
      }
      if (!released) co.release();
    }
    if (half == 1) {
      s_half[0][rl] = st.m;
      s_half[1][rl] = st.all;
      s_half[2][rl] = st.far;
    }
  }
  __syncthreads();
  const bool ok = s_abort == 0;
  if (warp >= 2 && half == 0) {
    // the two halves of every row meet
    const float m2 = s_half[0][rl], mn = fmaxf(st.m, m2);
    const float c1 = ex2(st.m - mn), c2 = ex2(m2 - mn);
    const float all = st.all * c1 + s_half[1][rl] * c2, far = st.far * c1 + s_half[2][rl] * c2;
    float ratio = (ok && row < p.N && all > 0.f) ? far / all : 0.f;
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) ratio += __shfl_xor_sync(0xffffffffu, ratio, o);
    if (lane == 0) s_ratio[quad] = ratio;
  }
  __syncthreads();
  if (tid == 0) {
    p.ratio_part[(size_t)unit * n_row_blocks + rb] = (s_ratio[0] + s_ratio[1]) + (s_ratio[2] + s_ratio[3]);
    if (!ok) atomicOr(p.status, 2u);
  }
  cta_teardown(tmem);
}

// ----------------------------------------------------------------------------- score
// The tiles of a scoring CTA, in the order all three roles walk them: for every block of 128
// observed queries, the key tiles of sweep 1 (from key 0) and then of sweep 2 (from the tile that
// holds the first image key), both up to the context of the block's last row.
struct ScoreBlock {
  int r0, last, ctx_max, k_first2;
};
// Block bi of n_blocks.  The blocks are aligned to the END of the observed queries: when their number is not a
// multiple of 128 it is the FIRST block that is short (rows [0, n_obs mod 128) of the tile loaded at row 0; the
// rows behind them belong to the next block and are left out like rows that do not exist), so the ragged block is
// the one with the shortest context and the fewest key tiles, not the one with the most.
__device__ __forceinline__ ScoreBlock score_block(const ScoreParams& p, int bi, int n_blocks) {
  ScoreBlock b;
  const int r_end = p.n_obs - (n_blocks - 1 - bi) * kRows;
  b.r0 = max(r_end - kRows, 0);
  b.last = r_end - 1;
  b.ctx_max = p.L + (p.n0 - p.n_obs + 1) + b.last;   // keys [0, ctx_max) are visible to the block's last row
  b.k_first2 = (p.L / kKeys) * kKeys;
  return b;
}

// Which of n_parts thread blocks takes query block b of a pair: dealt back and forth (0, 1, .., P-1, P-1, ..,
// 1, 0, 0, ..), so that every part gets short and long contexts alike.
__device__ __forceinline__ int block_owner(int b, int n_parts) {
  const int r = b % n_parts;
  return ((b / n_parts) & 1) ? n_parts - 1 - r : r;
}

// n_parts CTAs per (sequence, semantic head), each looping over its blocks of 128 observed queries; a
// part writes its own score row (zeros where it had nothing to add), and the selection adds the parts up
// in a fixed order.
__global__ void __launch_bounds__(kTcThreads, 2)
ssd_score_kernel(const ScoreParams p, const __grid_constant__ CUtensorMap tq, const __grid_constant__ CUtensorMap tk) {
  extern __shared__ __align__(1024) unsigned char smem[];
  __shared__ PipeBars s_bars;
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort;
  __shared__ float s_half[2][2][2][kRows];   // [block parity][column half][m, exp-sum][row]: sweep-1 statistics
  const int n_pairs = p.n_seqs * p.H;
  // the parts of a pair are neighbours in launch order, so they run at the same time and find each other's
  // key tiles in L2
  const int pair = blockIdx.x / p.n_parts, part = blockIdx.x % p.n_parts;
  const int head = pair % p.H;
  if (!p.desc[head].w) return;            // before any tensor-memory allocation
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int t_first = p.n0 - p.n_obs + 1;  // image step of observed row 0
  const int n_blocks = (p.n_obs + kRows - 1) / kRows;

  if (tid == 0) {                      // while the thread block sets itself up
    prefetch_map(&tq);
    prefetch_map(&tk);
  }
  Pipe pipe;
  // the two small operand tiles of the normalisers come first, so that whatever the tensor core reads through
  // their descriptors lies inside this thread block's own tiles
  const uint32_t ext_s = cta_setup(smem, s_bars, &s_tmem, &s_abort, pipe);
  const uint32_t q_s = ext_s + kExtBytes, k_s = q_s + kTileBytes;
  unsigned char* ext_p = smem + (ext_s - smem_u32(smem));
  const uint32_t tmem = s_tmem;

  if (warp == 0) {
    if (lane == 0) {
      Producer pr;
      pr.p = pipe; pr.abort = &s_abort; pr.q_s = q_s; pr.k_s = k_s; pr.tq = &tq; pr.tk = &tk;
      for (int bi = 0; bi < n_blocks; ++bi) {
        if (block_owner(bi, p.n_parts) != part) continue;
        const ScoreBlock b = score_block(p, bi, n_blocks);
        pr.query_block(b.r0, pair);
        for (int k0 = 0; k0 < b.ctx_max; k0 += kKeys) pr.key_tile(k0, pair);
        for (int k0 = b.k_first2; k0 < b.ctx_max; k0 += kKeys) pr.key_tile(k0, pair);
      }
      pr.drain();
    }
  } else if (warp == 1) {
    if (lane == 0) {
      Issuer is;
      is.p = pipe; is.abort = &s_abort; is.q_s = q_s; is.k_s = k_s; is.tmem = tmem; is.ext_s = ext_s;
      for (int bi = 0; bi < n_blocks; ++bi) {
        if (block_owner(bi, p.n_parts) != part) continue;
        const ScoreBlock b = score_block(p, bi, n_blocks);
        is.query_block();
        for (int k0 = 0; k0 < b.ctx_max; k0 += kKeys) is.key_tile();
        for (int k0 = b.k_first2; k0 < b.ctx_max; k0 += kKeys) is.key_tile(true, k0 == b.k_first2);
        is.end_block();
      }
    }
  } else {
    const int quad = warp & 3, half = (warp - 2) >> 2;   // TMEM lane quadrant; which half of a tile's columns
    const int rl = quad * 32 + lane;                     // row inside a block of queries
    Consumer co;
    co.p = pipe; co.abort = &s_abort; co.tmem_lane = tmem + ((uint32_t)(quad * 32) << 16); co.lane = lane;
    // this warp's score row in sweep 2: one per half of a block's queries; a key always belongs to the same lane
    float* my_score = p.score + ((((size_t)part * n_pairs + pair) * kScoreHalves) + half) * p.n0;

    if (half == 0) {
      // once: row rl of the tile of ones (1 in the three columns the normalisers use), and the upper half of
      // row rl of the tile of normalisers, which stays zero
      uint4* ones = reinterpret_cast<uint4*>(ext_p + ext_row_offset(rl));
      ones[0] = make_uint4(0x3f803f80u, 0x00003f80u, 0u, 0u);
      ones[8] = make_uint4(0u, 0u, 0u, 0u);
      reinterpret_cast<uint4*>(ext_p + kExtTileBytes + ext_row_offset(rl))[8] = make_uint4(0u, 0u, 0u, 0u);
    }
    const float inv_scale = 1.f / p.scale_log2;

    int blk = 0;                           // blocks this part has done
    for (int bi = 0; bi < n_blocks; ++bi) {
      if (block_owner(bi, p.n_parts) != part) continue;
      const ScoreBlock b = score_block(p, bi, n_blocks);
      const int r0 = b.r0;
      const int row = r0 + rl;
      const int ctx_r = row <= b.last ? p.L + t_first + row : 0;          // keys [0, ctx_r) are visible (none to rows left out)
      const int lo_row = r0 + quad * 32;
      const bool warp_full = lo_row + 31 <= b.last;                       // all 32 rows of the warp exist
      const int lo_ctx = p.L + t_first + lo_row;                          // context of the warp's first row
      // and of its last; 0 (nothing to do in either sweep) when the block ends before the warp's rows
      const int warp_ctx = lo_row <= b.last ? p.L + t_first + min(lo_row + 31, b.last) : 0;

      // sweep 1: row maximum and exp-sum
      RowStats st = {kNegBig, 0.f, 0.f};
      for (int k0 = 0; k0 < b.ctx_max; k0 += kKeys) {
        const uint32_t acc = co.tile();
        bool released = false;
#pragma unroll 1
        for (int cb = 2 * half; cb < 2 * half + 2; ++cb) {
          const int base = k0 + cb * 32;
          if (base >= warp_ctx) break;
          float v[32];
          tmem_ld32(acc + cb * 32, v);
          if (cb == 2 * half + 1) {
            co.release();
            released = true;
          }
          if (warp_full && base + 32 <= lo_ctx) fold32<false, false>(st, v, 32, 0, false, p.scale_log2);
          else fold32<true, false>(st, v, clamp32(ctx_r - base), 0, false, p.scale_log2);
        }
        if (!released) co.release();
      }
      // both threads of a row get the statistics of the whole row
      float (*xch)[2][kRows] = s_half[blk & 1];
      xch[half][0][rl] = st.m;
      xch[half][1][rl] = st.all;
      asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
      {
        const float m2 = xch[half ^ 1][0][rl], l2 = xch[half ^ 1][1][rl];
        const float mn = fmaxf(st.m, m2);
        // the same expression in both threads (operands ordered by column half), so they agree bit for bit
        const float lo_m = half ? m2 : st.m, hi_m = half ? st.m : m2;
        const float lo_l = half ? l2 : st.all, hi_l = half ? st.all : l2;
        st.all = lo_l * ex2(lo_m - mn) + hi_l * ex2(hi_m - mn);
        st.m = mn;
      }
      // the normaliser goes into the exponent: p = 2^(x - (m + log2 l)), one multiplication less per logit
      const float m_l = st.all > 0.f ? st.m + __log2f(st.all) : 1.0e30f;
      if (half == 0) {
        // -(m + log2 l) / scale as three bf16 terms (each remainder is exact in float32); rows that do not exist
        // get a large negative number, their columns are not read
        const float a = st.all > 0.f ? -m_l * inv_scale : -30000.f;
        const __nv_bfloat16 a1 = __float2bfloat16_rn(a);
        const float r1 = a - __bfloat162float(a1);
        const __nv_bfloat16 a2 = __float2bfloat16_rn(r1);
        const __nv_bfloat16 a3 = __float2bfloat16_rn(r1 - __bfloat162float(a2));
        const uint32_t w0 = (uint32_t)__bfloat16_as_ushort(a1) | ((uint32_t)__bfloat16_as_ushort(a2) << 16);
        const uint32_t w1 = (uint32_t)__bfloat16_as_ushort(a3);
        *reinterpret_cast<uint4*>(ext_p + kExtTileBytes + ext_row_offset(rl)) = make_uint4(w0, w1, 0u, 0u);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // before the tensor core reads it
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(pipe.ext_full());
      }

      // sweep 2, transposed tiles with the normalisers already subtracted: this thread is key k0 + rl of the tile
      // and sums that key's probabilities over the queries of its half of the block (two groups of 32 columns)
      const int row_ctx0 = p.L + t_first + r0;          // context of the block's first row; row r sees keys < row_ctx0 + r
      const int n_rows = b.last - r0 + 1;               // rows of the block that exist
      for (int k0 = b.k_first2; k0 < b.ctx_max; k0 += kKeys) {
        const uint32_t acc = co.tile();
        bool released = false;
        const int key_lo = k0 + quad * 32, key = key_lo + lane;
        float total = 0.f;
#pragma unroll 1
        for (int cb = 2 * half; cb < 2 * half + 2; ++cb) {
          const int q0 = cb * 32;                         // first row of this group, inside the block
          if (q0 >= n_rows) break;                        // the block ends before these rows
          if (key_lo + 32 <= p.L) break;                  // prompt keys only: not scored
          if (key_lo >= row_ctx0 + min(q0 + 31, n_rows - 1)) continue;   // no row of the group sees a key of this warp
          float v[32];
          tmem_ld32(acc + q0, v);
          if (cb == 2 * half + 1) {
            co.release();
            released = true;
          }
          float sum[4] = {0.f, 0.f, 0.f, 0.f};            // four chains of eight additions, joined in a fixed order
          if (q0 + 32 <= n_rows && key_lo + 32 <= row_ctx0 + q0) {      // every row exists and sees all 32 keys
#pragma unroll
            for (int j = 0; j < 32; ++j) sum[j & 3] += ex2(v[j] * p.scale_log2);
          } else {
            // row q0 + j sees this key iff key < row_ctx0 + q0 + j, and exists iff q0 + j < n_rows
            const int j_lo = max(key - row_ctx0 - q0 + 1, 0), j_hi = min(n_rows - q0, 32);
#pragma unroll
            for (int j = 0; j < 32; ++j) sum[j & 3] += (j >= j_lo && j < j_hi) ? ex2(v[j] * p.scale_log2) : 0.f;
          }
          total += (sum[0] + sum[1]) + (sum[2] + sum[3]);
        }
        if (!released) co.release();
        // an addition that returns nothing, so nothing waits for it; this lane is the only one that ever
        // adds to this element, and its additions arrive in program order: the sum is reproducible
        if (key >= p.L && key < b.ctx_max) atomicAdd(my_score + (key - p.L), total);
      }
      ++blk;
    }
  }

  __syncthreads();
  if (tid == 0 && s_abort != 0) atomicOr(p.status, 4u);    // the pair's rows are incomplete
  cta_teardown(tmem);
}

// ---- tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn tensor_map_encoder() {
  static EncodeTiledFn fn = [] {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q = cudaDriverEntryPointSymbolNotFound;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      f = nullptr;
    return reinterpret_cast<EncodeTiledFn>(f);
  }();
  return fn;
}

// Map of a [units, rows, 128] bf16 tensor, read in boxes of 128 rows x 64 elements with the 128-byte
// swizzle; rows past `rows` read as zeros.
cudaError_t make_tile_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t units) {
  EncodeTiledFn enc = tensor_map_encoder();
  if (!enc) return cudaErrorNotSupported;
  if (rows == 0 || units == 0 || rows >> 31 || units >> 31) return cudaErrorInvalidValue;
  const cuuint64_t dims[3] = {(cuuint64_t)kHeadDim, rows, units};
  const cuuint64_t strides[2] = {(cuuint64_t)kHeadDim * 2, rows * kHeadDim * 2};
  const cuuint32_t box[3] = {64, 128, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

}  // namespace

int classify_rows_per_block() { return kRows; }

cudaError_t launch_classify(const ClassifyParams& p, int n_row_blocks, cudaStream_t st) {
  const int smem = (1 + kStages) * kTileBytes + 1024;
  CUtensorMap tq, tk;
  cudaError_t e = make_tile_map(&tq, p.q_cal, (uint64_t)p.N, (uint64_t)p.n_units);
  if (e == cudaSuccess) e = make_tile_map(&tk, p.k_cal, (uint64_t)p.L + p.N, (uint64_t)p.n_units);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(ssd_classify_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  ssd_classify_kernel<<<p.n_units * n_row_blocks, kTcThreads, smem, st>>>(p, n_row_blocks, tq, tk);
  count_launch();
  return cudaGetLastError();
}

// Two scoring CTAs fit an SM.  With P parts per pair the launch needs ceil(pairs * P / slots) rounds of CTAs,
// each 1/P of a pair's work long: take the P that makes that product smallest (the smaller P on ties), as
// long as every part still gets at least two query blocks.
int score_parts(int n_sem_pairs, int n_obs) {
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
    cudaGetLastError();
    sms = 148;
  }
  const long slots = 2L * sms;
  const int n_blocks = (n_obs + kRows - 1) / kRows;
  int best = 1;
  double best_cost = 1e30;
  for (int parts = 1; parts <= kScoreMaxParts && 2 * parts <= (n_blocks > 2 ? n_blocks : 2); ++parts) {
    const long rounds = ((long)n_sem_pairs * parts + slots - 1) / slots;
    const double cost = (double)rounds / parts;
    if (cost < best_cost * (1.0 - 1e-9)) {
      best_cost = cost;
      best = parts;
    }
  }
  return best;
}

cudaError_t launch_score(const ScoreParams& p, cudaStream_t st) {
  const size_t smem = (1 + kStages) * (size_t)kTileBytes + kExtBytes + 1024;
  CUtensorMap tq, tk;
  const uint64_t pairs = (uint64_t)p.n_seqs * p.H;
  cudaError_t e = make_tile_map(&tq, p.q_obs, (uint64_t)p.n_obs, pairs);
  if (e == cudaSuccess) e = make_tile_map(&tk, p.k_full, (uint64_t)p.L + p.n0, pairs);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(ssd_score_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  if (p.n_parts < 1 || p.n_parts > kScoreMaxParts) return cudaErrorInvalidValue;
  ssd_score_kernel<<<p.n_seqs * p.H * p.n_parts, kTcThreads, smem, st>>>(p, tq, tk);
  count_launch();
  return cudaGetLastError();
}

}  // namespace ssd
