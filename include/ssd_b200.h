/*
 * ssd_b200.h -- C ABI of the SSD head-decoupled compressed KV cache for single-token
 * decode attention on NVIDIA B200 (sm_100a).
 *
 * The method (paper: "SSD: Spatial-Semantic Head Decoupling for Efficient Autoregressive
 * Image Generation") splits attention heads into spatial-locality heads, which keep a short
 * window of the most recent visual tokens, and semantic-sink heads, which keep the top-M
 * visual tokens by accumulated attention score plus a small reserved recent window
 * (Sec. 3.3, Algorithm 1).  This library holds that cache and runs attention over it.
 *
 * Conventions
 *  - All tensors are bf16, row-major, innermost dimension head_dim (= 128).
 *  - Pointers named *_host are host memory; every other data pointer is DEVICE memory owned
 *    by the caller.  The library allocates no device memory: the caller hands one device
 *    buffer to ssd_cache_create and it is carved up internally.
 *  - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Calls enqueue work
 *    on it and return; exceptions are noted per function.  One cache must be driven from one
 *    stream at a time (launches that overlap on the GPU would race on its scratch areas).
 *  - Host threads: a cache is not synchronised; calls on the SAME cache must not overlap in time
 *    (its host state, e.g. the token counters, is plain data).  Calls on DIFFERENT caches may run
 *    on different host threads concurrently: what they share (the per-device set-up of the kernels'
 *    shared-memory limits, the launch counter, the fixed array of ssd_decode_attn_static) is set
 *    up or updated atomically.  Every call acts on the calling thread's current device, which must
 *    be the device that holds the cache's buffer.
 *  - L = prompt_len prompt tokens are retained whole by every head.  Image token j (0-based)
 *    has absolute position L + j; image step t = j + 1.  The "initial sink token" that Sec. 3.3
 *    keeps beside the window of a spatial head is position 0, i.e. the first prompt token, which
 *    is retained with the prompt; with prompt_len = 0 there is no such token and a spatial head
 *    keeps exactly its W newest image tokens.
 *  - All sequences advance in lock step: every call acts on all n_seqs sequences of a layer.
 *  - Every function returns an ssd_status (0 = SSD_OK, negative = error) unless noted; all
 *    argument checking happens on the host before anything is launched.
 */
#ifndef SSD_B200_H
#define SSD_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ssd_cache ssd_cache; /* opaque; created by ssd_cache_create, owned by the library */

typedef struct ssd_config {
  int32_t n_layers;
  int32_t n_seqs;           /* sequences (a classifier-free-guidance pair is two) */
  int32_t n_heads;          /* multi-head attention: kv heads == query heads; <= 128 */
  int32_t head_dim;         /* must be 128 */
  int32_t prompt_len;       /* L >= 0 */
  int32_t max_image_tokens; /* N = h*w of the token grid */
  int32_t window;           /* W >= 1: ring slots of a spatial head, newest token included */
  int32_t sink_budget;      /* M >= 0: top-M static slots of a semantic head */
  int32_t sink_recent;      /* R >= 1: ring slots of a semantic head, newest token included */
  int32_t cls_window;       /* w of the sparsity metric (Sec. 3.3; the paper uses 32) */
  float tau;                /* a head is semantic iff its sparsity s > tau (Sec. 3.3) */
  float softmax_scale;      /* 0 selects 1/sqrt(head_dim) */
} ssd_config;

enum ssd_status {
  SSD_OK = 0,
  SSD_ERR_INVALID_ARG = -1, /* null pointer, out-of-range size or layer */
  SSD_ERR_BAD_STATE = -2,   /* call order violated (e.g. compress before labels exist) */
  SSD_ERR_OVERFLOW = -3,    /* append beyond max_image_tokens (cf. Algorithm 2, buffer overflow) */
  SSD_ERR_NO_MEM = -4,      /* caller's device buffer too small for the layout */
  SSD_ERR_CUDA = -5,        /* a CUDA runtime call or launch failed */
  SSD_ERR_LIMIT = -6        /* a size exceeds a fixed limit of the entry point called */
};

/* Human-readable name of a status code (static storage; never NULL). */
const char *ssd_status_string(int status);

/* Device bytes ssd_cache_create needs.  n_sink_heads_total = number of (layer, head) entries
 * that will be labelled semantic; pass -1 for the worst case over all labelings.  Returns 0 on
 * an invalid config. */
size_t ssd_cache_required_bytes(const ssd_config *cfg, int32_t n_sink_heads_total);

/* Create a cache over caller-owned device memory [dev_mem, dev_mem + dev_bytes) (256-byte
 * aligned).  The config carries what Algorithm 1 lists as its parameters (window size, token budget) and
 * what Sec. 3.3 adds (reserved recent window, threshold).  Validates the config, lays out tables and scratch at the front of the buffer and
 * clears them (synchronously, on the default stream).  Head labels do not exist yet: call
 * ssd_classify_heads or ssd_set_head_labels next.  The buffer must outlive the cache. */
int ssd_cache_create(const ssd_config *cfg, void *dev_mem, size_t dev_bytes, ssd_cache **out);

/* Release the host object.  The device buffer stays with the caller.  NULL is accepted. */
int ssd_cache_free(ssd_cache *cache);

/* Head classification (Sec. 3.3): sparsity s[l,h] = mean over calibration sequences p and image
 * steps t of (attention mass on visual tokens older than the newest cls_window) / (mass on all
 * visual tokens so far); label = s > tau.
 *   q_cal [n_layers, n_cal_seqs, n_heads, n_img, head_dim]   queries of image steps 1..n_img
 *   k_cal [n_layers, n_cal_seqs, n_heads, prompt_len + n_img, head_dim]
 *     (device, bf16, dense, 16-byte aligned: read by the TMA unit; SSD_ERR_INVALID_ARG otherwise)
 *   s_out_host      [n_layers * n_heads] float  (may be NULL)
 *   labels_out_host [n_layers * n_heads] uint8, 1 = semantic (may be NULL)
 * Installs the labels in the cache (fixing the per-head layout) and SYNCHRONISES the stream.
 * SSD_ERR_NO_MEM if the resulting layout does not fit the buffer. */
int ssd_classify_heads(ssd_cache *cache, const void *q_cal, const void *k_cal, int32_t n_cal_seqs,
                       int32_t n_img, float *s_out_host, uint8_t *labels_out_host, void *stream);

/* The same measurement without installing labels: writes, per (layer, head), the sum over the
 * given calibration sequences and steps of the ratio above (double, [n_layers * n_heads]).  A
 * caller that shards calibration sequences over several GPUs adds these sums across ranks,
 * divides by (total sequences * n_img) and calls ssd_set_head_labels.  Synchronises the stream. */
int ssd_classify_partial(ssd_cache *cache, const void *q_cal, const void *k_cal, int32_t n_cal_seqs,
                         int32_t n_img, double *ratio_sums_host, void *stream);

/* The threshold rule of Sec. 3.3 on its own, for callers that hold ratio sums (ssd_classify_partial,
 * added over ranks) or sparsity values (a sweep of tau, Sec. 4.3/4.4).  Host arithmetic only; no GPU and
 * no cache is needed.
 *   ssd_labels_from_ratio_sums: s[i] = (float)(ratio_sums[i] / (n_cal_total * n_img)), label[i] = s[i] > tau
 *     (equality is spatial), exactly what ssd_classify_heads computes; s_out_host and labels_out_host
 *     [n] may each be NULL.
 *   ssd_labels_from_sparsity:   label[i] = s[i] > tau for float32 sparsity values.
 * SSD_ERR_INVALID_ARG on null inputs, n < 0, non-finite tau, n_cal_total < 1 or n_img < 1. */
int ssd_labels_from_ratio_sums(const double *ratio_sums_host, int64_t n, int32_t n_cal_total, int32_t n_img,
                               float tau, float *s_out_host, uint8_t *labels_out_host);
int ssd_labels_from_sparsity(const float *s_host, int64_t n, float tau, uint8_t *labels_out_host);

/* Install head labels directly ([n_layers * n_heads] uint8, 1 = semantic): what a caller that shards
 * the calibration batch does after ssd_labels_from_ratio_sums (Sec. 3.3), and how by-construction or
 * random partitions are set (Sec. 4.4 ablation).  Resets every layer to the empty state. */
int ssd_set_head_labels(ssd_cache *cache, const uint8_t *labels_host);

/* Bulk-load one layer from an uncompressed cache holding the prompt and n0 image tokens, and
 * compress it (Algorithm 1; Algorithm 2's prefill split when n0 == 0).
 *   q_obs  [n_seqs, n_heads, n_obs, head_dim]  queries of image steps n0-n_obs+1 .. n0
 *   k_full, v_full [n_seqs, n_heads, prompt_len + n0, head_dim]
 *     (device, bf16, dense, 16-byte aligned; SSD_ERR_INVALID_ARG otherwise)
 * Semantic heads: score[j] = sum over the observed steps of the post-softmax attention on image
 * token j (causal, softmax over prompt + image tokens); keep the min(M, n0-R) best-scoring
 * tokens among j in [0, n0-R) (ties: lowest j), stored in ascending j, plus the R newest tokens.
 * Spatial heads: keep the W newest tokens.  Every head keeps the whole prompt.
 * 0 <= n0 <= max_image_tokens; 0 <= n_obs <= n0 (q_obs may be NULL when n_obs == 0 or the layer
 * has no semantic head).  Replaces the layer's previous contents.  Asynchronous.
 * Should a bounded wait of the scoring kernel run out, the scores of that pair are incomplete and bit 2
 * of the device status word is set (ssd_cache_device_status): check it after compressing when the
 * selection matters. */
int ssd_compress(ssd_cache *cache, int32_t layer, const void *q_obs, const void *k_full,
                 const void *v_full, int32_t n0, int32_t n_obs, void *stream);

/* Append the newest token's K/V for every (sequence, head) of a layer: written into the head's
 * ring, overwriting (evicting) the oldest ring entry once the ring is full (Algorithm 1, Append).
 *   k_new, v_new [n_seqs, n_heads, head_dim], 16-byte aligned (SSD_ERR_INVALID_ARG otherwise: the
 *   kernel reads them 16 bytes at a time)
 * SSD_ERR_OVERFLOW once max_image_tokens tokens are held.  Asynchronous. */
int ssd_append(ssd_cache *cache, int32_t layer, const void *k_new, const void *v_new, void *stream);

/* Single-token decode attention (Sec. 3.1, the attention of one generated token over the cached keys and
 * values; the caches are Algorithm 1's output, its Ensure line) over the layer's retained slots, both
 * head types in one launch:
 * out[s,h] = sum_i softmax_i(scale * <q[s,h], K_i>) V_i over the prompt, static and ring slots
 * that hold a token (the token just appended included).  fp32 accumulation, bf16 output.
 *   q, out [n_seqs, n_heads, head_dim], 16-byte aligned
 * SSD_ERR_BAD_STATE if some head of the layer holds no token at all (no prompt loaded and, for that
 * head's type, nothing in its static set or ring): attention over nothing has no value.  Asynchronous. */
int ssd_decode_attn(ssd_cache *cache, int32_t layer, const void *q, void *out, void *stream);

/* ssd_append followed by ssd_decode_attn for the same layer, in one kernel launch (Algorithm 1's
 * Append and the attention that consumes its output).  Same arguments, results and errors as the two
 * calls; the newest token's rows are read from k_new / v_new by the attention and stored into the
 * ring by the same kernel.  k_new, v_new, q, out 16-byte aligned.  In row-buffer mode (below) it is still
 * one launch: the kernel keeps the step's logits in one of two alternating buffers and, at its start, adds
 * the weights of the layer's previous step to the scores (which nothing reads in between but
 * ssd_recompress and ssd_cache_get_scores, and those add what is pending themselves).  Asynchronous. */
int ssd_append_decode(ssd_cache *cache, int32_t layer, const void *k_new, const void *v_new,
                      const void *q, void *out, void *stream);

/* ssd_append_decode for n_layers consecutive layers in ONE launch (a whole decode step when the
 * inputs of all layers exist up front, as in a benchmark of this path or a host-driven replay; in a
 * model, layer l+1's query depends on layer l's output and the per-layer call is the one to use).
 *   k_new, v_new, q, out [n_layers, n_seqs, n_heads, head_dim] bf16 on the device, 16-byte
 *   aligned; entry i belongs to layer first_layer + i.
 * Results are those of the per-layer call up to the rounding order of the softmax sums (a head is
 * summed by one warp here, by up to several there).  The work is handed out head by head from a
 * counter in the cache buffer, so the layers need not have the same layout or occupancy.
 * In row-buffer mode (Algorithm 2) the kernel also adds the step's attention weights to the scores
 * of semantic heads (a head is summed by one warp, which therefore holds all its weights), so
 * nothing is left pending for the next append or ssd_recompress; the per-layer calls and this one
 * can be mixed freely.
 * With a row buffer of one token (sink_recent = 1) the launch re-selects too, which is Algorithm 1
 * taken literally: after the step's attention the token just appended takes the place of the
 * lowest-scoring static token (or a still unused static slot), or is dropped itself if its own
 * score is the lowest (ties: the highest position leaves); the buffer is empty again when the call
 * returns and ssd_recompress has nothing left to do.
 * SSD_ERR_LIMIT if n_layers > 64 (issue several calls) or, in row-buffer mode, if sink_budget +
 * sink_recent exceeds what a warp can keep in shared memory (about 3000; 1000 with
 * sink_recent = 1); SSD_ERR_OVERFLOW (nothing launched) if any of the layers, or its row buffer,
 * is full.  Asynchronous. */
int ssd_append_decode_layers(ssd_cache *cache, int32_t first_layer, int32_t n_layers, const void *k_new,
                             const void *v_new, const void *q, void *out, void *stream);

/* Row-buffer mode (Algorithm 2, Appendix B).  With the mode on, the ring of a semantic head is the
 * algorithm's row buffer of R = sink_recent tokens, filled from empty:
 *   ssd_compress     selects the top-M over all n0 tokens (the buffer starts empty) and records the
 *                    selected tokens' scores;
 *   ssd_append       puts the token into the buffer; SSD_ERR_OVERFLOW when the buffer already holds R
 *                    tokens (Algorithm 2, overflow branch): call ssd_recompress first;
 *   ssd_decode_attn  attends over prompt + static set + buffer and keeps the step's attention weights
 *                    of the static and buffered tokens of semantic heads; they are added to the tokens'
 *                    accumulated scores by the layer's next ssd_append or ssd_recompress;
 *   ssd_recompress   (Algorithm 2, buffer-full branch): per (sequence, semantic head) keeps the top-M of static set +
 *                    buffer by accumulated score (ties: lowest position) as the new static set and
 *                    empties the buffer.  Tokens that stay keep their slots; tokens that enter take
 *                    the slots of those that leave, so static slots are in ascending position only
 *                    until the first re-selection.  Asynchronous.
 * Spatial heads keep exactly their W newest tokens in both modes.  ssd_cache_set_row_buffer switches the
 * mode and resets every layer to the empty state (call it before ssd_compress).
 * ssd_cache_get_scores: acc_host [n_seqs, n_heads, M + R] accumulated scores, entry e < M for static
 * slot e, entry M + r for buffer slot r, including the last decode's weights; -1 for entries that hold no
 * token or belong to spatial heads.  Synchronises the device. */
int ssd_cache_set_row_buffer(ssd_cache *cache, int32_t enable);
int ssd_recompress(ssd_cache *cache, int32_t layer, void *stream);
/* ssd_recompress for n_layers consecutive layers in one launch (same results, layer by layer): with
 * ssd_append_decode_layers, a buffer cycle of Algorithm 2 is R + 1 launches for all layers.  Layers
 * with an empty buffer and nothing pending are skipped (no launch at all if that is all of them).
 * With sink_recent = 1 (Algorithm 1 taken literally: a re-selection after every step) no ranking is needed
 * and a lighter kernel, one warp per (sequence, head), drops the lowest score; same results.
 * SSD_ERR_LIMIT if n_layers > 64. */
int ssd_recompress_layers(ssd_cache *cache, int32_t first_layer, int32_t n_layers, void *stream);
int ssd_cache_get_scores(ssd_cache *cache, int32_t layer, float *acc_host);

/* The accumulated scores the latest ssd_compress computed (Algorithm 1, AttentionScores summed over the
 * observed steps), before selection: score_host [n_seqs, n_heads, n0] float, -1 for spatial heads.
 * The scores live in a buffer that every ssd_compress and ssd_classify_* call reuses, so this works only
 * for the layer compressed last (SSD_ERR_BAD_STATE otherwise, or if that call needed no scores).
 * For inspection and parity; synchronises the device. */
int ssd_cache_get_compress_scores(ssd_cache *cache, int32_t layer, float *score_host);

/* ssd_decode_attn for callers that cannot allocate.  The paper has no counterpart; this is a
 * packaging variant of the same kernel.  ssd_decode_attn keeps the kernel's scratch (partial sums of
 * heads that two thread blocks share, and per-head arrival counters) inside the buffer given to
 * ssd_cache_create.  Some callers have no memory to give beyond their tensors and cannot call
 * cudaMalloc where they stand: code running between the capture calls of a stream, plugins inside a
 * host program that owns all device memory through its own pool, or real-time loops in which an
 * allocation's implicit synchronisation is not acceptable.  For them the same scratch is a fixed
 * array inside the library image (about 0.4 MB, held by every GPU that loads the library until the
 * process ends), and this call allocates nothing, on the device or through any library.
 *   Same arguments, results and errors as ssd_decode_attn (outputs are bit-identical), plus
 *   SSD_ERR_LIMIT if n_seqs * n_heads > 32768 or the GPU has more than 256 SMs: the array is sized
 *   for those maxima.
 * The first call on each device looks up the array's device address (a synchronous runtime query);
 * make that first call before any stream capture begins.  All calls on a device share the one
 * array, whatever cache they pass: two calls whose kernels overlap on the GPU (different streams)
 * race on it; calls on one stream are safe.  The counters are cleared on `stream` at every call,
 * the partials are always written before they are read.  Bounded-wait failures are reported in the
 * cache's status word like those of ssd_decode_attn. */
int ssd_decode_attn_static(ssd_cache *cache, int32_t layer, const void *q, void *out, void *stream);

/* 8-bit K/V.  The paper does not quantise; it cites quantisation as the orthogonal line of work (Sec. 2, "KV
 * Cache Compression").  This is that extension on the same head-decoupled store: every cached row is held as
 * 128 E4M3 codes (OCP 8-bit floating point: 4 exponent bits, bias 7, 3 mantissa bits, largest magnitude 448) and
 * one float32 scale per row, scale = max|x| / 448, code = E4M3(x / scale) with round to nearest even, saturating,
 * decided in float32 arithmetic; a slot is 272 bytes instead of 512.  A row is quantised once, when it enters the
 * cache.  Attention runs in float32 on the exactly widened codes; the K row's scale multiplies the logit, the V
 * row's the softmax weight.
 *   ssd_cache_set_kv_format(cache, 1) switches a cache to that format (0 = bf16, the default) and resets every
 *   layer to the empty state; call it before ssd_compress.  In that format the cache serves ssd_compress,
 *   ssd_append_decode_layers, ssd_append_decode and ssd_decode_attn (the equal-shares kernel of the bf16 path
 *   with this format's arithmetic), ssd_step_host(_layers) and the inspection calls; ssd_append (a row is
 *   quantised by the launch that first attends to it), ssd_decode_attn_static and the row-buffer mode return
 *   SSD_ERR_BAD_STATE (so does switching the format while the row buffer is on, and vice versa).  The device buffer
 *   is sized as for bf16 (ssd_cache_required_bytes); ssd_cache_kv_bytes reports the bytes actually held.
 *   ssd_quantize_rows_e4m3 is the quantiser on its own: rows [n_rows, 128] bf16 -> codes_out [n_rows, 128] uint8 and
 *   scales_out [n_rows] float (all on the device; rows and codes_out 16-byte aligned).  Asynchronous. */
int ssd_cache_set_kv_format(ssd_cache *cache, int32_t format);
int ssd_quantize_rows_e4m3(const void *rows, int64_t n_rows, void *codes_out, float *scales_out, void *stream);

/* Per-token divergence of two KV caches (Sec. 3.2, the MSE_token equation; the paper compares the cache of
 * the guided branch with that of the native branch of one prompt, position by position):
 *   mse_out[r] = ||k_a[r] - k_b[r]||^2 + ||v_a[r] - v_b[r]||^2,  r = 0 .. n_rows-1
 * where a row is one token of one head: k_a, v_a, k_b, v_b [n_rows, head_dim = 128] bf16 on the device,
 * dense, 16-byte aligned (any leading shape, e.g. [n_seqs, n_heads, tokens], flattened); mse_out [n_rows]
 * float on the device.  The sum is as printed: no division by head_dim.  fp32 arithmetic on the exactly
 * widened inputs.  Needs no cache.  SSD_ERR_INVALID_ARG on null or misaligned pointers or n_rows < 0;
 * n_rows = 0 does nothing.  Asynchronous. */
int ssd_kv_token_mse(const void *k_a, const void *v_a, const void *k_b, const void *v_b, int64_t n_rows,
                     float *mse_out, void *stream);

/* One decode step of one layer from HOST buffers (pinned memory recommended): copies q, k_new and
 * v_new to the device, appends, attends, and copies the output back, all enqueued on `stream`.
 *   q_host, k_new_host, v_new_host, out_host [n_seqs, n_heads, head_dim] bf16 on the host
 * The host buffers must stay untouched until the stream has drained.  Asynchronous. */
int ssd_step_host(ssd_cache *cache, int32_t layer, const void *q_host, const void *k_new_host,
                  const void *v_new_host, void *out_host, void *stream);

/* The same for n_layers consecutive layers in one call, with the copies running beside the kernels:
 * layers move in groups of 10 (one copy per tensor and group); a group's inputs are copied on a
 * stream of the library's own while the group before it is attended to, and its outputs go back
 * on another while the next group runs (a ring of 3 staging slots inside the cache buffer; the
 * streams and events are created at the first call).
 *   q_host, k_new_host, v_new_host, out_host [n_layers, n_seqs, n_heads, head_dim] bf16 on the
 *   host, pinned (pageable memory works but serialises the copies); entry i belongs to layer
 *   first_layer + i.
 * The kernels are ordered after the work already on `stream`, and `stream` is made to wait for the
 * last copy, so the results are on the host once `stream` has drained; until then the host buffers
 * must stay untouched.  The INPUT copies do not wait for earlier work on `stream` (so that the next
 * step's inputs travel under this step's kernels): the input buffers must hold their values when
 * the call is made.  SSD_ERR_OVERFLOW (nothing enqueued) if any of the layers is full.
 * Asynchronous. */
int ssd_step_host_layers(ssd_cache *cache, int32_t first_layer, int32_t n_layers, const void *q_host,
                         const void *k_new_host, const void *v_new_host, void *out_host, void *stream);

/* Absolute positions held by each slot of a layer (the index sets Algorithm 1 keeps: IndicesOfTopM for
 * semantic heads, the last W for spatial heads), for inspection and index-set parity:
 * idx_host [n_seqs, n_heads, max_slots] int32 with max_slots = ssd_cache_max_slots(); slots are
 * ordered prompt, static (ascending position after ssd_compress; slot order after re-selections
 * in row-buffer mode), ring (physical ring order); -1 = empty or unused.
 * Synchronises the device. */
int ssd_cache_get_indices(ssd_cache *cache, int32_t layer, int32_t *idx_host);
int32_t ssd_cache_max_slots(const ssd_cache *cache); /* prompt_len + max(window, M + R) */

/* Number of slots currently holding a token, per head of a layer: len_host [n_heads]. */
int ssd_cache_get_lengths(ssd_cache *cache, int32_t layer, int32_t *len_host);

/* Current labels ([n_layers * n_heads] uint8) and image tokens held so far by a layer. */
int ssd_cache_get_labels(ssd_cache *cache, uint8_t *labels_host);
int32_t ssd_cache_tokens(const ssd_cache *cache, int32_t layer); /* -1 on bad arguments */

/* Set a layer's image-token counter back to an earlier value t (n0 <= t <= current), so a
 * benchmark can replay the same decode steps; ring contents are not restored. */
int ssd_cache_rewind(ssd_cache *cache, int32_t layer, int32_t t);

/* K+V bytes the cache holds per sequence over all layers at full occupancy (slots * 512 B). */
int ssd_cache_kv_bytes(ssd_cache *cache, size_t *bytes_per_seq);

/* Device-side timing of decode launches, for measurement.  ssd_profile_enable creates CUDA events
 * for up to max_launches launches (0 switches timing off); while enabled, every ssd_decode_attn
 * records an event before and after its kernel on the caller's stream.  ssd_profile_collect waits
 * for the recorded launches, writes their durations in milliseconds to ms_host (room for
 * max_launches floats), their number to *n_out, and starts over.  No paper counterpart. */
int ssd_profile_enable(ssd_cache *cache, int32_t max_launches);
int ssd_profile_collect(ssd_cache *cache, float *ms_host, int32_t *n_out);

/* Device status word of the cache (0 = healthy).  Every wait inside a kernel is limited to about a
 * second; a kernel that gives one up sets a bit here and finishes without the missing data:
 *   bit 0 (1): a decode warp (ssd_decode_attn, ssd_append_decode, ssd_append_decode_layers,
 *              ssd_decode_attn_static) gave up waiting for one of its asynchronous copies or for a partial
 *              result; the outputs of that launch are incomplete;
 *   bit 1 (2): the classifier (ssd_classify_heads / ssd_classify_partial) gave up; its sparsity values
 *              are incomplete;
 *   bit 2 (4): the scoring kernel of ssd_compress gave up; the scores of the affected pairs are
 *              incomplete, and so is the selection made from them.
 * The bits are sticky until the cache is recreated.  The kernels never trap and never spin without a
 * limit, so the CUDA context stays usable.  Synchronises the device.  No paper counterpart. */
int ssd_cache_device_status(ssd_cache *cache, uint32_t *status_host);

/* Inspection of the decode kernel's work decomposition, computed on the host by the same code the
 * kernel runs (no GPU needed): lists every bulk copy one ssd_decode_attn launch would issue for a
 * layer with the given per-head layout and occupancy.
 *   head_recs [n_heads][4] = {first slot of the head inside a sequence's block, static capacity,
 *             ring capacity, 1 if semantic}; heads are packed back to back (prompt_len + static
 *             + ring slots each)
 *   prompt_valid 0 or prompt_len; static_valid valid top-M slots of semantic heads; t_img image
 *   tokens held; max_workers warps available; chunk slots per copy stage (0 = the kernel's own)
 *   copies_out [cap][6] = {worker, chunk number within the worker, source slot (from the layer's
 *             first slot), destination slot within the stage, slots copied, sequence*n_heads+head}
 * Copies are listed in stream order per worker; the kernel issues the same copies, except that a
 * worker whose last head runs past its thread block's range starts with that head's piece.
 * Returns the number of copies (which may exceed cap; only the first cap are written) or a negative
 * ssd_status.  No paper counterpart. */
int64_t ssd_debug_decode_plan(int32_t n_heads, const int32_t *head_recs, int32_t prompt_len,
                              int32_t n_seqs, int32_t prompt_valid, int32_t static_valid,
                              int32_t t_img, int32_t max_workers, int32_t chunk,
                              int64_t *copies_out, int64_t cap);

/* Number of kernels this library has launched since the process started (for audit). */
uint64_t ssd_kernel_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* SSD_B200_H */
