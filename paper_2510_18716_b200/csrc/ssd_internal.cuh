// Internal declarations shared by the translation units of the SSD B200 library.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "ssd_b200.h"
#include "ssd_plan.h"

namespace ssd {

constexpr int kHeadDim = 128;
constexpr int kSlotBytes = 512;          // one token of one head: K row (256 B) then V row (256 B)
constexpr int kSlotU4 = kSlotBytes / 16; // 32 uint4 per slot
constexpr int kMaxHeads = 128;
constexpr int kPartialFloats = 132;      // m, l, 2 pad, acc[128]

// Per (layer, head) layout record, resident in device memory.
//   x = slot offset of the head inside one sequence's block of the layer
//   y = static capacity (M for semantic heads, 0 for spatial)
//   z = ring capacity (R for semantic heads, W for spatial)
//   w = 1 for semantic heads
typedef int4 HeadDesc;

struct DecodeParams {
  const uint4* slab;        // first slot of the layer
  const __nv_bfloat16* q;   // [n_seqs, H, 128]
  __nv_bfloat16* out;       // [n_seqs, H, 128]
  float* partial;           // [max workers * 2, kPartialFloats]
  uint32_t* counters;       // [n_seqs * H], zero between launches
  uint32_t* status;         // device status word (bit 0: a bounded wait ran out)
  float* logits;            // row-buffer mode: [n_seqs * H, M + R] logits (base 2) of the static and
                            // ring slots of semantic heads, for the score accumulation; else null
  float2* ml;               // row-buffer mode: [n_seqs * H] final (max, exp-sum) of each head; else null
  int mr;                   // M + R
  // fused append: the newest token's rows are not in the slab yet (null / -1 when it is)
  const unsigned char* k_new;  // [n_seqs, H, 128] bf16: K row of image token new_j
  const unsigned char* v_new;
  int new_j;                // image index of that token; the view already counts it
  int sem_slot;             // row-buffer mode: buffer slot of that token in semantic heads; else -1 (slot new_j mod R)
  // Row-buffer mode, fused append (Algorithm 2, score accumulation, one launch per step and layer): before
  // anything else the launch brings the scores up to date with the layer's PREVIOUS decode, whose logits
  // and (max, exp-sum) are in fold_logits / fold_ml (the other of two alternating buffers, so that this
  // launch's own logits do not overwrite them), and starts the new token's score at zero.  fold_acc ==
  // nullptr: nothing to do.
  float* fold_acc;          // [n_seqs * H, M + R]
  const float* fold_logits; // [n_seqs * H, M + R]; read only if fold_pending
  const float2* fold_ml;    // [n_seqs * H]
  int fold_pending;         // 1: the previous decode's weights are not yet in the scores
  int fold_static, fold_buffered;   // static and buffered entries that held a token at that decode
  int early;                // 1: the launch before this one on the stream does not write this layer's slab
  float scale_log2;         // softmax scale * log2(e)
  Split split;              // how the layer's slots are shared out (set by launch_decode)
  LayerView view;           // layout and occupancy of the layer
};

// One launch for a whole step (every layer's fused append + decode).
constexpr int kMaxLayersPerLaunch = 64;
struct LayerState {
  long long first_slot;     // the layer's first slot in the slab
  const HeadDesc* desc;     // [H] layout records of the layer (device)
  int seq_slots;            // physical slots per sequence
  int prompt_valid;         // 0 or L
  int static_valid;         // valid static slots of semantic heads
  int t_img;                // image tokens held, the one being appended included
  int new_j;                // image index of the token being appended
  // row-buffer mode (Algorithm 2): the rings of semantic heads are buffers filled from slot 0
  int t_sem;                // tokens in those buffers, the one being appended included
  int sem_slot;             // buffer slot of the token being appended
};
struct DecodeLayersParams {
  uint4* slab;              // slot 0 of the slab
  const unsigned char* q;   // [n_layers, n_seqs, H, 128] bf16
  const unsigned char* k_new;
  const unsigned char* v_new;
  __nv_bfloat16* out;       // [n_layers, n_seqs, H, 128]
  uint32_t* status;         // device status word (bit 0: a bounded wait ran out)
  uint32_t* work;           // next unit to hand out; zero at launch
  int n_layers, n_seqs, H, L;
  // row-buffer mode (Algorithm 2); acc == nullptr outside it.  A layer's tables follow the previous
  // layer's at fixed strides, so the first layer's pointers serve all.
  float* acc;               // first layer's [n_seqs * H, M + R] accumulated attention scores
  int32_t* static_idx;      // first layer's [n_seqs, H, M] image indices of the static slots
  int M;                    // static capacity of semantic heads
  int mr;                   // M + R: entries of a head's score row
  int evict;                // 1 (R == 1 only): the launch also re-selects, i.e. the token just appended
                            // takes the place of the lowest-scoring static token, or is dropped itself
  float scale_log2;
  LayerState layer[kMaxLayersPerLaunch];
};

struct AppendParams {
  uint4* slab;
  const HeadDesc* desc;
  const uint4* k_new;       // [n_seqs, H, 16] uint4
  const uint4* v_new;
  int n_seqs, H, L;
  int j;                    // image index of the token being appended
  int seq_slots;
  // row-buffer mode (Algorithm 2); acc == nullptr otherwise
  int sem_slot;             // ring slot of semantic heads for this token (tokens buffered so far)
  int static_valid;         // valid static slots of semantic heads
  int pending;              // 1: the logits of the layer's last decode are not yet in the scores
  int mr;                   // M + R
  float* acc;               // [n_seqs * H, M + R] accumulated attention scores
  const float* logits;      // [n_seqs * H, M + R]
  const float2* ml;         // [n_seqs * H]
};

struct GatherParams {
  uint4* slab;
  const HeadDesc* desc;
  int sem_ring;              // 0: leave the rings of semantic heads empty (row-buffer mode)
  const int32_t* static_idx; // [n_seqs, H, M] image indices, ascending, -1 padded
  const uint4* k_full;       // [n_seqs, H, L + n0, 16] uint4
  const uint4* v_full;
  int n_seqs, H, L, M, n0;
  int static_valid;
  int seq_slots;
  int after_select;          // 1: launched as the programmatic dependent of the selection kernel: the slots that
                             // do not hold selected tokens are copied while the selection may still be running
};

#if defined(__CUDACC__)
// Does slot s of a head hold a token chosen by the selection (a static slot of a semantic head)?
__device__ __forceinline__ bool gather_slot_selected(const GatherParams& p, const HeadDesc& d, int s) {
  return d.w && s >= p.L && s < p.L + d.y;
}
// Row of k_full / v_full that belongs in slot s of a head; -1: the slot stays empty.
__device__ __forceinline__ int gather_source_row(const GatherParams& p, const HeadDesc& d, int pair, int s) {
  if (s < p.L) return s;
  if (s < p.L + d.y) {
    const int mm = s - p.L;
    if (!d.w || mm >= p.static_valid) return -1;
    const int j = p.static_idx[(size_t)pair * p.M + mm];
    return (j >= 0 && j < p.n0) ? p.L + j : -1;
  }
  const int r = s - p.L - d.y;                   // ring slot r holds the newest j = r (mod capacity)
  if (p.n0 - 1 >= r && (p.sem_ring || !d.w)) return p.L + ((p.n0 - 1 - r) / d.z) * d.z + r;
  return -1;
}
#endif

struct ScoreParams {
  const __nv_bfloat16* q_obs;  // [n_seqs, H, n_obs, 128]
  const __nv_bfloat16* k_full; // [n_seqs, H, L + n0, 128]
  const HeadDesc* desc;
  float* score;                // [n_parts][n_seqs, H][2][n0], zero at launch: row (part, pair, half) gets the sums
                               // over that half of the query rows of the query blocks of that part
  uint32_t* status;            // device status word (bit 2: a bounded wait of the scoring ran out)
  int n_seqs, H, L, n0, n_obs;
  int n_parts;                 // thread blocks that share the query blocks of one (sequence, head)
  float scale_log2;
};

struct SelectParams {
  float* score;                // [n_parts][n_seqs, H][2][n0]; a pair's 2 * n_parts rows are first added, in a
                               // fixed order, into its row (part 0, half 0), which is the pair's score row
  int n_parts;
  const HeadDesc* desc;
  int32_t* static_idx;         // [n_seqs, H, M]
  float* acc;                  // row-buffer mode: [n_seqs * H, mr], gets the selected tokens' scores; else null
  int mr;
  int n_seqs, H, M, n0, n_cand;
};

struct ClassifyParams {
  const __nv_bfloat16* q_cal;  // [n_units, N, 128], unit = (layer, p, head)
  const __nv_bfloat16* k_cal;  // [n_units, L + N, 128]
  float* ratio_part;           // [n_units, n_row_blocks]
  uint32_t* status;            // device status word (bit 1: a bounded wait of the classifier ran out)
  int n_units, L, N, w;
  float scale_log2;
};

cudaError_t launch_decode(const DecodeParams& p, cudaStream_t st);
cudaError_t launch_decode_layers(const DecodeLayersParams& p, cudaStream_t st);
// acc += the normalised weights of the layer's last decode (its logits and (max, exp-sum) are in
// `logits` and `ml`): what the next append of the row-buffer mode would do first
cudaError_t launch_fold_pending(float* acc, const float* logits, const float2* ml, const HeadDesc* desc, int n_seqs,
                                int H, int mr, int static_valid, int buffered, cudaStream_t st);
int decode_layers_max_mr();
cudaError_t launch_append(const AppendParams& p, cudaStream_t st);
cudaError_t launch_gather(const GatherParams& p, int max_slots, cudaStream_t st);
cudaError_t launch_score(const ScoreParams& p, cudaStream_t st);
constexpr int kScoreMaxParts = 4;
constexpr int kScoreHalves = 2;  // score rows a scoring thread block keeps per pair: one per half of a block's queries
int score_parts(int n_sem_pairs, int n_obs);   // thread blocks per (sequence, head) the scoring kernel should use
cudaError_t launch_select(const SelectParams& p, cudaStream_t st);
struct RecompressParams {
  uint4* slab;
  const HeadDesc* desc;
  int32_t* static_idx;         // [n_seqs, H, M] image indices of the static slots (updated)
  float* acc;                  // [n_seqs * H, mr] accumulated scores (updated)
  const float* logits;         // pending logits of the last decode
  const float2* ml;
  int pending;
  int n_seqs, H, L, M, mr;
  int static_valid;            // valid static slots before the call
  int buffered;                // tokens in the row buffer
  int t_base;                  // image index of the buffer's first token
  int seq_slots;
};
cudaError_t launch_recompress(const RecompressParams& p, cudaStream_t st);
// 8-bit K/V (slots of 272 bytes: 128 + 128 E4M3 codes and two float32 row scales)
cudaError_t launch_quantize_rows(const void* rows, long long n_rows, void* codes, float* scales, cudaStream_t st);
cudaError_t launch_gather_q8(const GatherParams& p, int max_slots, cudaStream_t st);
cudaError_t launch_decode_layers_q8(const DecodeLayersParams& p, cudaStream_t st);
cudaError_t launch_decode_q8(const DecodeParams& p, cudaStream_t st);   // one layer, 8-bit slots (no row-buffer fields)
int q8_slot_bytes();
// The same for several layers in one launch: what differs from layer to layer, and the first layer's
// tables (a layer's tables follow the previous layer's at fixed strides).
struct RecompressLayer {
  long long first_slot;        // the layer's first slot in the slab
  int seq_slots, static_valid, buffered, t_base, pending;
  int lg;                      // which of the layer's two logit buffers holds the pending logits
  int todo;                    // 0: nothing buffered and nothing pending in this layer
};
struct RecompressLayersParams {
  uint4* slab;                 // slot 0 of the slab
  const HeadDesc* desc;        // first layer's [H] records; next layer H records further
  int32_t* static_idx;         // first layer's [n_seqs, H, M]
  float* acc;                  // first layer's [n_seqs * H, mr]
  const float* logits;         // first layer's first buffer; two buffers per layer
  const float2* ml;
  int n_layers, n_seqs, H, L, M, mr;
  RecompressLayer layer[kMaxLayersPerLaunch];
};
cudaError_t launch_recompress_layers(const RecompressLayersParams& p, cudaStream_t st);
// the same for a row buffer of one token (every layer has at most one token buffered): one warp per pair
cudaError_t launch_evict_one_layers(const RecompressLayersParams& p, cudaStream_t st);
cudaError_t launch_classify(const ClassifyParams& p, int n_row_blocks, cudaStream_t st);
int classify_rows_per_block();
int decode_max_workers();
int decode_chunk_slots();

void count_launch(int n = 1);

}  // namespace ssd
