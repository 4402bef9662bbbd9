// Host side of the C ABI: argument checking, the per-head variable-length layout, per-layer
// state, and the sequencing of kernels.  No device memory is allocated here: everything lives in
// the buffer the caller passed to ssd_cache_create.
#include <atomic>
#include <cmath>
#include <cstring>
#include <new>

#include "ssd_internal.cuh"

namespace ssd {

static std::atomic<uint64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

static size_t align_up(size_t x, size_t a = 256) { return (x + a - 1) / a * a; }

// ssd_step_host_layers moves layers in groups of kHostGroup (one copy per tensor and group: a copy
// of one layer's 0.5 MB costs about as much in set-up as in transfer) through a ring of kHostSlots
// staging slots; a slot holds q, k_new, v_new and out of a whole group.
constexpr int kHostGroup = 10;
constexpr int kHostSlots = 3;

struct Regions {
  size_t desc, idx, counters, status, partial, score, staging, acc, logits, ml, slab;  // byte offsets
  size_t score_bytes, partial_bytes, front_bytes;
};

static bool config_ok(const ssd_config* c) {
  if (!c) return false;
  if (c->n_layers < 1 || c->n_seqs < 1 || c->n_heads < 1 || c->n_heads > kMaxHeads) return false;
  if (c->head_dim != kHeadDim) return false;
  if (c->prompt_len < 0 || c->max_image_tokens < 1) return false;
  if (c->window < 1 || c->sink_budget < 0 || c->sink_recent < 1) return false;
  if (c->cls_window < 0) return false;
  if (!(c->softmax_scale >= 0.f) || !std::isfinite(c->softmax_scale)) return false;
  if (!std::isfinite(c->tau)) return false;
  // keep every index in 32 bits with room to spare
  const double slots = (double)c->prompt_len + std::fmax((double)c->window, (double)c->sink_budget + c->sink_recent);
  if (slots * c->n_heads > 1.0e9 || (double)c->n_seqs * c->n_heads > 5.0e8) return false;
  if (slots * c->n_heads * c->n_seqs > 2.0e9) return false;   // slots of one layer are counted in 32 bits
  if ((double)c->prompt_len + c->max_image_tokens > 1.0e8) return false;
  return true;
}

static Regions plan_regions(const ssd_config& c) {
  Regions r;
  size_t off = 0;
  const size_t pairs_layer = (size_t)c.n_seqs * c.n_heads;
  r.desc = off;      off = align_up(off + (size_t)c.n_layers * c.n_heads * sizeof(HeadDesc));
  r.idx = off;       off = align_up(off + (size_t)c.n_layers * pairs_layer * (c.sink_budget > 0 ? c.sink_budget : 1) * 4);
  r.counters = off;  off = align_up(off + pairs_layer * 4);
  r.status = off;    off = align_up(off + 132);   // status word, and at +128 the unit counter of the all-layers launch
  r.partial_bytes = (size_t)decode_max_workers() * 2 * kPartialFloats * 4;
  r.partial = off;   off = align_up(off + r.partial_bytes);
  // scoring: two rows (one per half of the query rows) for every thread block that shares a pair's query blocks
  r.score_bytes = pairs_layer * (size_t)c.max_image_tokens * 4 * kScoreHalves * kScoreMaxParts;
  r.score = off;     off = align_up(off + r.score_bytes);
  r.staging = off;   off = align_up(off + (size_t)kHostSlots * kHostGroup * 4 * pairs_layer * kHeadDim * 2);
  // row-buffer mode (Algorithm 2): accumulated scores and the last decode's logits of the static and
  // ring slots, and the last decode's (max, exp-sum), per layer
  const size_t mr = (size_t)c.sink_budget + c.sink_recent;
  r.acc = off;       off = align_up(off + (size_t)c.n_layers * pairs_layer * mr * 4);
  // two buffers per layer each: a launch that records a step's logits may, at its start, still be adding
  // those of the step before to the scores
  r.logits = off;    off = align_up(off + (size_t)c.n_layers * 2 * pairs_layer * mr * 4);
  r.ml = off;        off = align_up(off + (size_t)c.n_layers * 2 * pairs_layer * 8);
  r.front_bytes = off;
  r.slab = off;
  return r;
}

}  // namespace ssd

using namespace ssd;

struct ssd_cache {
  ssd_config cfg;
  float scale;
  char* base;
  size_t bytes;
  Regions reg;
  bool labels_set;
  std::vector<uint8_t> labels;        // [layers*H]
  std::vector<HeadDesc> desc;         // [layers*H]
  std::vector<int32_t> seq_slots;     // [layers]
  std::vector<int64_t> layer_base;    // [layers] first slot of the layer in the slab
  std::vector<int32_t> n_sink;        // [layers]
  std::vector<int32_t> t_img, n0, prompt_valid, static_valid;  // [layers]
  // Layer whose slab the library's latest launch may write (append, fused append, compress,
  // re-selection), -1 if none, -2 if unknown: a decode launch of ANOTHER layer may prefetch its slab
  // before that launch has completed.
  int last_writer = -2;
  int score_layer = -1, score_n0 = 0; // layer whose prefill scores (ssd_compress) the score buffer holds, -1 if none
  bool row_buffer = false;            // Algorithm 2: rings of semantic heads are row buffers
  std::vector<int32_t> t_base;        // [layers] image tokens held when the buffer was last emptied
  std::vector<uint8_t> pending;       // [layers] last decode's logits not yet added to the scores
  std::vector<uint8_t> lg_cur;        // [layers] which of the layer's two logit buffers the last decode wrote
  // ssd_step_host_layers: copy streams and per-slot events, created at its first call
  cudaStream_t h_in = nullptr, h_out = nullptr;
  cudaEvent_t h_fork = nullptr, h_loaded[kHostSlots] = {}, h_done[kHostSlots] = {}, h_stored[kHostSlots] = {};
  long h_groups = 0;                  // groups sent through the staging ring so far
  bool h_foreign = false;             // ssd_step_host has used the staging area since
  std::vector<cudaEvent_t> prof_ev;   // 2 events per timed decode launch (empty = timing off)
  int prof_n = 0;                     // launches recorded since the last collect

  HeadDesc* d_desc(int layer) const { return reinterpret_cast<HeadDesc*>(base + reg.desc) + (size_t)layer * cfg.n_heads; }
  int32_t* d_idx(int layer) const {
    size_t per = (size_t)cfg.n_seqs * cfg.n_heads * (cfg.sink_budget > 0 ? cfg.sink_budget : 1);
    return reinterpret_cast<int32_t*>(base + reg.idx) + (size_t)layer * per;
  }
  uint32_t* d_counters() const { return reinterpret_cast<uint32_t*>(base + reg.counters); }
  uint32_t* d_status() const { return reinterpret_cast<uint32_t*>(base + reg.status); }
  uint32_t* d_work() const { return reinterpret_cast<uint32_t*>(base + reg.status + 128); }   // unit counter of the all-layers launch
  int mr() const { return cfg.sink_budget + cfg.sink_recent; }
  size_t layer_scores(int layer) const { return (size_t)layer * cfg.n_seqs * cfg.n_heads * mr(); }
  float* d_acc(int layer) const { return reinterpret_cast<float*>(base + reg.acc) + layer_scores(layer); }
  float* d_logits(int layer, int which) const {
    return reinterpret_cast<float*>(base + reg.logits) + ((size_t)layer * 2 + which) * cfg.n_seqs * cfg.n_heads * mr();
  }
  float2* d_ml(int layer, int which) const {
    return reinterpret_cast<float2*>(base + reg.ml) + ((size_t)layer * 2 + which) * cfg.n_seqs * cfg.n_heads;
  }
  // tokens in the rings of semantic heads
  int sem_tokens(int layer) const { return row_buffer ? t_img[layer] - t_base[layer] : t_img[layer]; }
  float* d_partial() const { return reinterpret_cast<float*>(base + reg.partial); }
  float* d_score() const { return reinterpret_cast<float*>(base + reg.score); }
  char* d_staging(int slot = 0) const {
    return base + reg.staging + (size_t)slot * kHostGroup * 4 * cfg.n_seqs * cfg.n_heads * kHeadDim * 2;
  }
  bool kv_q8 = false;                 // 8-bit K/V: slots of 272 bytes (E4M3 codes and row scales) instead of 512
  int slot_bytes() const { return kv_q8 ? q8_slot_bytes() : kSlotBytes; }
  uint4* d_slab(int layer) const {
    return reinterpret_cast<uint4*>(base + reg.slab + (size_t)layer_base[layer] * slot_bytes());
  }
  int max_slots() const {
    int a = cfg.window, b = cfg.sink_budget + cfg.sink_recent;
    return cfg.prompt_len + (a > b ? a : b);
  }
  // True if some head of the layer would hold no token at all with t image tokens in the layer (t_sem of
  // them in the rings of semantic heads): attention over nothing has no value, so decode refuses.
  bool empty_head(int layer, int t, int t_sem) const {
    if (prompt_valid[layer] > 0) return false;
    if (n_sink[layer] < cfg.n_heads && t == 0) return true;                               // a spatial head
    return n_sink[layer] > 0 && static_valid[layer] == 0 && t_sem == 0;                   // a semantic head
  }
  // layout and occupancy of a layer, as the decode kernel sees it
  void fill_view(int layer, LayerView& v) const {
    v.H = cfg.n_heads; v.L = cfg.prompt_len; v.n_seqs = cfg.n_seqs; v.seq_slots = seq_slots[layer];
    v.prompt_valid = prompt_valid[layer];
    v.static_valid = static_valid[layer];
    v.t_img = t_img[layer];
    v.t_sem = sem_tokens(layer);
    for (int h = 0; h < cfg.n_heads; ++h) {
      const HeadDesc& d = desc[(size_t)layer * cfg.n_heads + h];
      v.head[h] = HeadRec{d.x, d.y, d.z, d.w};
    }
    view_finish(v);
  }
};

static size_t slab_slots_for(const ssd_config& c, long n_sink_total) {
  const long heads_total = (long)c.n_layers * c.n_heads;
  const size_t spatial = (size_t)c.prompt_len + c.window;
  const size_t sink = (size_t)c.prompt_len + c.sink_budget + c.sink_recent;
  if (n_sink_total < 0) return (size_t)heads_total * (spatial > sink ? spatial : sink) * c.n_seqs;
  return ((size_t)n_sink_total * sink + (size_t)(heads_total - n_sink_total) * spatial) * c.n_seqs;
}

extern "C" {

const char* ssd_status_string(int s) {
  switch (s) {
    case SSD_OK: return "SSD_OK";
    case SSD_ERR_INVALID_ARG: return "SSD_ERR_INVALID_ARG";
    case SSD_ERR_BAD_STATE: return "SSD_ERR_BAD_STATE";
    case SSD_ERR_OVERFLOW: return "SSD_ERR_OVERFLOW";
    case SSD_ERR_NO_MEM: return "SSD_ERR_NO_MEM";
    case SSD_ERR_CUDA: return "SSD_ERR_CUDA";
    case SSD_ERR_LIMIT: return "SSD_ERR_LIMIT";
    default: return "SSD_ERR_UNKNOWN";
  }
}

uint64_t ssd_kernel_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

size_t ssd_cache_required_bytes(const ssd_config* cfg, int32_t n_sink_heads_total) {
  if (!config_ok(cfg)) return 0;
  if (n_sink_heads_total > cfg->n_layers * cfg->n_heads) return 0;
  Regions r = plan_regions(*cfg);
  return r.front_bytes + slab_slots_for(*cfg, n_sink_heads_total) * kSlotBytes;
}

int ssd_cache_create(const ssd_config* cfg, void* dev_mem, size_t dev_bytes, ssd_cache** out) {
  if (!out) return SSD_ERR_INVALID_ARG;
  *out = nullptr;
  if (!config_ok(cfg) || !dev_mem) return SSD_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(dev_mem) % 256 != 0) return SSD_ERR_INVALID_ARG;
  Regions r = plan_regions(*cfg);
  // at least the all-spatial or all-semantic layout, whichever is smaller, must fit
  size_t a = slab_slots_for(*cfg, 0), b = slab_slots_for(*cfg, (long)cfg->n_layers * cfg->n_heads);
  if (dev_bytes < r.front_bytes + (a < b ? a : b) * kSlotBytes) return SSD_ERR_NO_MEM;
  ssd_cache* c = new (std::nothrow) ssd_cache();
  if (!c) return SSD_ERR_NO_MEM;
  c->cfg = *cfg;
  c->scale = cfg->softmax_scale > 0.f ? cfg->softmax_scale : 1.0f / std::sqrt((float)cfg->head_dim);
  c->base = static_cast<char*>(dev_mem);
  c->bytes = dev_bytes;
  c->reg = r;
  c->labels_set = false;
  const size_t nh = (size_t)cfg->n_layers * cfg->n_heads;
  c->labels.assign(nh, 0);
  c->desc.assign(nh, HeadDesc{0, 0, 0, 0});
  c->seq_slots.assign(cfg->n_layers, 0);
  c->layer_base.assign(cfg->n_layers, 0);
  c->n_sink.assign(cfg->n_layers, 0);
  c->t_img.assign(cfg->n_layers, 0);
  c->n0.assign(cfg->n_layers, 0);
  c->prompt_valid.assign(cfg->n_layers, 0);
  c->static_valid.assign(cfg->n_layers, 0);
  c->t_base.assign(cfg->n_layers, 0);
  c->pending.assign(cfg->n_layers, 0);
  c->lg_cur.assign(cfg->n_layers, 0);
  if (cudaMemset(c->base, 0, r.front_bytes) != cudaSuccess ||
      cudaMemset(c->base + r.idx, 0xFF, r.counters - r.idx) != cudaSuccess ||
      cudaDeviceSynchronize() != cudaSuccess) {
    cudaGetLastError();
    delete c;
    return SSD_ERR_CUDA;
  }
  *out = c;
  return SSD_OK;
}

static void destroy_events(ssd_cache* c) {
  for (cudaEvent_t e : c->prof_ev) cudaEventDestroy(e);
  c->prof_ev.clear();
  c->prof_n = 0;
}

static void destroy_host_pipe(ssd_cache* c) {
  if (c->h_in) cudaStreamDestroy(c->h_in);
  if (c->h_out) cudaStreamDestroy(c->h_out);
  if (c->h_fork) cudaEventDestroy(c->h_fork);
  for (int i = 0; i < kHostSlots; ++i) {
    if (c->h_loaded[i]) cudaEventDestroy(c->h_loaded[i]);
    if (c->h_done[i]) cudaEventDestroy(c->h_done[i]);
    if (c->h_stored[i]) cudaEventDestroy(c->h_stored[i]);
    c->h_loaded[i] = c->h_done[i] = c->h_stored[i] = nullptr;
  }
  c->h_in = c->h_out = nullptr;
  c->h_fork = nullptr;
}

static bool make_host_pipe(ssd_cache* c) {
  if (c->h_in) return true;
  bool ok = cudaStreamCreateWithFlags(&c->h_in, cudaStreamNonBlocking) == cudaSuccess &&
            cudaStreamCreateWithFlags(&c->h_out, cudaStreamNonBlocking) == cudaSuccess &&
            cudaEventCreateWithFlags(&c->h_fork, cudaEventDisableTiming) == cudaSuccess;
  for (int i = 0; ok && i < kHostSlots; ++i)
    ok = cudaEventCreateWithFlags(&c->h_loaded[i], cudaEventDisableTiming) == cudaSuccess &&
         cudaEventCreateWithFlags(&c->h_done[i], cudaEventDisableTiming) == cudaSuccess &&
         cudaEventCreateWithFlags(&c->h_stored[i], cudaEventDisableTiming) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    destroy_host_pipe(c);
  }
  return ok;
}

int ssd_cache_free(ssd_cache* c) {
  if (c) destroy_events(c);
  if (c) destroy_host_pipe(c);
  delete c;
  return SSD_OK;
}

int ssd_profile_enable(ssd_cache* c, int32_t max_launches) {
  if (!c || max_launches < 0) return SSD_ERR_INVALID_ARG;
  destroy_events(c);
  for (int i = 0; i < 2 * max_launches; ++i) {
    cudaEvent_t e;
    if (cudaEventCreate(&e) != cudaSuccess) {
      cudaGetLastError();
      destroy_events(c);
      return SSD_ERR_CUDA;
    }
    c->prof_ev.push_back(e);
  }
  return SSD_OK;
}

int ssd_profile_collect(ssd_cache* c, float* ms_host, int32_t* n_out) {
  if (!c || !ms_host || !n_out) return SSD_ERR_INVALID_ARG;
  for (int i = 0; i < c->prof_n; ++i) {
    if (cudaEventSynchronize(c->prof_ev[2 * i + 1]) != cudaSuccess ||
        cudaEventElapsedTime(ms_host + i, c->prof_ev[2 * i], c->prof_ev[2 * i + 1]) != cudaSuccess) {
      cudaGetLastError();
      return SSD_ERR_CUDA;
    }
  }
  *n_out = c->prof_n;
  c->prof_n = 0;
  return SSD_OK;
}

int ssd_set_head_labels(ssd_cache* c, const uint8_t* labels_host) {
  if (!c || !labels_host) return SSD_ERR_INVALID_ARG;
  const ssd_config& g = c->cfg;
  const size_t nh = (size_t)g.n_layers * g.n_heads;
  long n_sink_total = 0;
  for (size_t i = 0; i < nh; ++i) n_sink_total += labels_host[i] ? 1 : 0;
  if (c->reg.front_bytes + slab_slots_for(g, n_sink_total) * kSlotBytes > c->bytes) return SSD_ERR_NO_MEM;
  std::vector<HeadDesc> desc(nh);
  int64_t base = 0;
  for (int l = 0; l < g.n_layers; ++l) {
    int off = 0, ns = 0;
    for (int h = 0; h < g.n_heads; ++h) {
      const bool sem = labels_host[(size_t)l * g.n_heads + h] != 0;
      HeadDesc d;
      d.x = off;
      d.y = sem ? g.sink_budget : 0;
      d.z = sem ? g.sink_recent : g.window;
      d.w = sem ? 1 : 0;
      desc[(size_t)l * g.n_heads + h] = d;
      off += g.prompt_len + d.y + d.z;
      ns += sem;
    }
    c->seq_slots[l] = off;
    c->layer_base[l] = base;
    c->n_sink[l] = ns;
    base += (int64_t)off * g.n_seqs;
  }
  if (cudaMemcpy(c->base + c->reg.desc, desc.data(), nh * sizeof(HeadDesc), cudaMemcpyHostToDevice) != cudaSuccess) {
    cudaGetLastError();
    return SSD_ERR_CUDA;
  }
  c->desc.swap(desc);
  for (size_t i = 0; i < nh; ++i) c->labels[i] = labels_host[i] ? 1 : 0;
  for (int l = 0; l < g.n_layers; ++l) {
    c->t_img[l] = c->n0[l] = c->prompt_valid[l] = c->static_valid[l] = c->t_base[l] = 0;
    c->pending[l] = 0;
  }
  c->labels_set = true;
  return SSD_OK;
}

int ssd_classify_partial(ssd_cache* c, const void* q_cal, const void* k_cal, int32_t n_cal_seqs, int32_t n_img,
                         double* ratio_sums_host, void* stream) {
  if (!c || !q_cal || !k_cal || !ratio_sums_host) return SSD_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(q_cal) | reinterpret_cast<uintptr_t>(k_cal)) % 16 != 0) return SSD_ERR_INVALID_ARG;
  const ssd_config& g = c->cfg;
  if (n_cal_seqs < 1 || n_img < 1 || n_img > g.max_image_tokens) return SSD_ERR_INVALID_ARG;
  const int rpb = classify_rows_per_block();
  const int nrb = (n_img + rpb - 1) / rpb;
  const size_t units = (size_t)g.n_layers * n_cal_seqs * g.n_heads;
  if (units * nrb * sizeof(float) > c->reg.score_bytes || units * nrb > 0x7fffffffULL) return SSD_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ClassifyParams p;
  p.q_cal = static_cast<const __nv_bfloat16*>(q_cal);
  p.k_cal = static_cast<const __nv_bfloat16*>(k_cal);
  p.ratio_part = c->d_score();
  p.status = c->d_status();
  p.n_units = (int)units;
  p.L = g.prompt_len;
  p.N = n_img;
  p.w = g.cls_window;
  p.scale_log2 = c->scale * 1.4426950408889634f;
  c->score_layer = -1;                 // the partial sums share the score buffer
  if (launch_classify(p, nrb, st) != cudaSuccess) return SSD_ERR_CUDA;
  std::vector<float> part(units * nrb);
  if (cudaMemcpyAsync(part.data(), c->d_score(), part.size() * sizeof(float), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess) {
    cudaGetLastError();
    return SSD_ERR_CUDA;
  }
  for (int l = 0; l < g.n_layers; ++l)
    for (int h = 0; h < g.n_heads; ++h) {
      double acc = 0.0;
      for (int pp = 0; pp < n_cal_seqs; ++pp) {
        const size_t unit = ((size_t)l * n_cal_seqs + pp) * g.n_heads + h;
        for (int rb = 0; rb < nrb; ++rb) acc += (double)part[unit * nrb + rb];
      }
      ratio_sums_host[(size_t)l * g.n_heads + h] = acc;
    }
  return SSD_OK;
}

// The threshold rule (Sec. 3.3): s = mean ratio, taken in float32; a head is semantic iff s > tau, so
// equality is spatial.  Host arithmetic only.
int ssd_labels_from_sparsity(const float* s_host, int64_t n, float tau, uint8_t* labels_out_host) {
  if (!s_host || !labels_out_host || n < 0 || !std::isfinite(tau)) return SSD_ERR_INVALID_ARG;
  for (int64_t i = 0; i < n; ++i) labels_out_host[i] = s_host[i] > tau ? 1 : 0;
  return SSD_OK;
}

int ssd_labels_from_ratio_sums(const double* ratio_sums_host, int64_t n, int32_t n_cal_total, int32_t n_img, float tau,
                               float* s_out_host, uint8_t* labels_out_host) {
  if (!ratio_sums_host || n < 0 || n_cal_total < 1 || n_img < 1 || !std::isfinite(tau)) return SSD_ERR_INVALID_ARG;
  for (int64_t i = 0; i < n; ++i) {
    const float s = (float)(ratio_sums_host[i] / ((double)n_cal_total * (double)n_img));
    if (s_out_host) s_out_host[i] = s;
    if (labels_out_host) ssd_labels_from_sparsity(&s, 1, tau, labels_out_host + i);
  }
  return SSD_OK;
}

int ssd_classify_heads(ssd_cache* c, const void* q_cal, const void* k_cal, int32_t n_cal_seqs, int32_t n_img,
                       float* s_out_host, uint8_t* labels_out_host, void* stream) {
  if (!c) return SSD_ERR_INVALID_ARG;
  const size_t nh = (size_t)c->cfg.n_layers * c->cfg.n_heads;
  std::vector<double> sums(nh);
  int rc = ssd_classify_partial(c, q_cal, k_cal, n_cal_seqs, n_img, sums.data(), stream);
  if (rc != SSD_OK) return rc;
  std::vector<uint8_t> lab(nh);
  rc = ssd_labels_from_ratio_sums(sums.data(), (int64_t)nh, n_cal_seqs, n_img, c->cfg.tau, s_out_host, lab.data());
  if (rc != SSD_OK) return rc;
  rc = ssd_set_head_labels(c, lab.data());
  if (rc != SSD_OK) return rc;
  if (labels_out_host) std::memcpy(labels_out_host, lab.data(), nh);
  return SSD_OK;
}

int ssd_compress(ssd_cache* c, int32_t layer, const void* q_obs, const void* k_full, const void* v_full, int32_t n0,
                 int32_t n_obs, void* stream) {
  if (!c || !k_full || !v_full) return SSD_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(q_obs) | reinterpret_cast<uintptr_t>(k_full) | reinterpret_cast<uintptr_t>(v_full)) % 16 != 0)
    return SSD_ERR_INVALID_ARG;
  const ssd_config& g = c->cfg;
  if (layer < 0 || layer >= g.n_layers) return SSD_ERR_INVALID_ARG;
  if (n0 < 0 || n0 > g.max_image_tokens || n_obs < 0 || n_obs > n0) return SSD_ERR_INVALID_ARG;
  if (!c->labels_set) return SSD_ERR_BAD_STATE;
  if (g.prompt_len + n0 < 1) return SSD_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the R newest tokens stay in the ring and are not candidates; with a row buffer (Algorithm 2,
  // prefill) the buffer starts empty and every token is a candidate
  const int n_cand = c->row_buffer ? n0 : (n0 - g.sink_recent > 0 ? n0 - g.sink_recent : 0);
  const int sv = g.sink_budget < n_cand ? g.sink_budget : n_cand;
  const bool select = c->n_sink[layer] > 0 && sv > 0;
  if (select && n_obs > 0 && !q_obs) return SSD_ERR_INVALID_ARG;
  c->score_layer = -1;
  const HeadDesc* desc = c->d_desc(layer);
  const int n_parts = (select && n_obs > 0) ? score_parts(g.n_seqs * c->n_sink[layer], n_obs) : 1;
  if (select) {
    if (n_obs > 0) {
      ScoreParams sp;
      sp.q_obs = static_cast<const __nv_bfloat16*>(q_obs);
      sp.k_full = static_cast<const __nv_bfloat16*>(k_full);
      sp.desc = desc;
      sp.score = c->d_score();
      sp.status = c->d_status();
      sp.n_seqs = g.n_seqs; sp.H = g.n_heads; sp.L = g.prompt_len; sp.n0 = n0; sp.n_obs = n_obs;
      sp.scale_log2 = c->scale * 1.4426950408889634f;
      sp.n_parts = n_parts;
      if (cudaMemsetAsync(c->d_score(), 0, (size_t)n_parts * g.n_seqs * g.n_heads * kScoreHalves * n0 * 4, st) != cudaSuccess ||
          launch_score(sp, st) != cudaSuccess) {
        cudaGetLastError();
        return SSD_ERR_CUDA;
      }
    } else {
      if (cudaMemsetAsync(c->d_score(), 0, (size_t)g.n_seqs * g.n_heads * kScoreHalves * n0 * 4, st) != cudaSuccess) return SSD_ERR_CUDA;
    }
    SelectParams sl;
    sl.score = c->d_score();
    sl.n_parts = n_parts;
    sl.desc = desc;
    sl.static_idx = c->d_idx(layer);
    sl.acc = c->row_buffer ? c->d_acc(layer) : nullptr;
    sl.mr = c->mr();
    sl.n_seqs = g.n_seqs; sl.H = g.n_heads; sl.M = g.sink_budget; sl.n0 = n0; sl.n_cand = n_cand;
    if (launch_select(sl, st) != cudaSuccess) return SSD_ERR_CUDA;
    c->score_layer = layer;
    c->score_n0 = n0;
  }
  GatherParams gp;
  gp.slab = c->d_slab(layer);
  gp.desc = desc;
  gp.static_idx = c->d_idx(layer);
  gp.sem_ring = c->row_buffer ? 0 : 1;
  gp.k_full = static_cast<const uint4*>(k_full);
  gp.v_full = static_cast<const uint4*>(v_full);
  gp.n_seqs = g.n_seqs; gp.H = g.n_heads; gp.L = g.prompt_len; gp.M = g.sink_budget; gp.n0 = n0;
  gp.static_valid = select ? sv : 0;
  gp.seq_slots = c->seq_slots[layer];
  gp.after_select = select ? 1 : 0;
  if ((c->kv_q8 ? launch_gather_q8(gp, c->max_slots(), st) : launch_gather(gp, c->max_slots(), st)) != cudaSuccess)
    return SSD_ERR_CUDA;
  c->t_img[layer] = n0;
  c->n0[layer] = n0;
  c->prompt_valid[layer] = g.prompt_len;
  c->static_valid[layer] = select ? sv : 0;
  c->t_base[layer] = n0;
  c->pending[layer] = 0;
  c->last_writer = -2;
  return SSD_OK;
}

int ssd_append(ssd_cache* c, int32_t layer, const void* k_new, const void* v_new, void* stream) {
  if (!c || !k_new || !v_new) return SSD_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(k_new) | reinterpret_cast<uintptr_t>(v_new)) % 16 != 0) return SSD_ERR_INVALID_ARG;
  const ssd_config& g = c->cfg;
  if (layer < 0 || layer >= g.n_layers) return SSD_ERR_INVALID_ARG;
  if (!c->labels_set || c->kv_q8) return SSD_ERR_BAD_STATE;   // 8-bit caches append inside the decode launch only
  if (c->t_img[layer] >= g.max_image_tokens) return SSD_ERR_OVERFLOW;
  if (c->row_buffer && c->n_sink[layer] > 0 && c->sem_tokens(layer) >= g.sink_recent)
    return SSD_ERR_OVERFLOW;            // Algorithm 2, overflow branch: call ssd_recompress first
  AppendParams p;
  p.slab = c->d_slab(layer);
  p.desc = c->d_desc(layer);
  p.k_new = static_cast<const uint4*>(k_new);
  p.v_new = static_cast<const uint4*>(v_new);
  p.n_seqs = g.n_seqs; p.H = g.n_heads; p.L = g.prompt_len;
  p.j = c->t_img[layer];
  p.seq_slots = c->seq_slots[layer];
  p.sem_slot = c->sem_tokens(layer);
  p.static_valid = c->static_valid[layer];
  p.pending = c->pending[layer];
  p.mr = c->mr();
  p.acc = c->row_buffer ? c->d_acc(layer) : nullptr;
  p.logits = c->d_logits(layer, c->lg_cur[layer]);
  p.ml = c->d_ml(layer, c->lg_cur[layer]);
  if (launch_append(p, static_cast<cudaStream_t>(stream)) != cudaSuccess) return SSD_ERR_CUDA;
  c->last_writer = layer;
  if (c->row_buffer) c->pending[layer] = 0;
  c->t_img[layer] += 1;
  return SSD_OK;
}

int ssd_decode_attn(ssd_cache* c, int32_t layer, const void* q, void* out, void* stream) {
  if (!c || !q || !out) return SSD_ERR_INVALID_ARG;
  const ssd_config& g = c->cfg;
  if (layer < 0 || layer >= g.n_layers) return SSD_ERR_INVALID_ARG;
  if (!c->labels_set) return SSD_ERR_BAD_STATE;
  if (c->empty_head(layer, c->t_img[layer], c->sem_tokens(layer))) return SSD_ERR_BAD_STATE;
  if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(out)) % 16 != 0) return SSD_ERR_INVALID_ARG;
  DecodeParams p;
  p.slab = c->d_slab(layer);
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.out = static_cast<__nv_bfloat16*>(out);
  p.partial = c->d_partial();
  p.counters = c->d_counters();
  p.status = c->d_status();
  const int lg_next = c->lg_cur[layer] ^ 1;
  p.logits = c->row_buffer ? c->d_logits(layer, lg_next) : nullptr;
  p.ml = c->row_buffer ? c->d_ml(layer, lg_next) : nullptr;
  p.mr = c->mr();
  p.k_new = nullptr; p.v_new = nullptr; p.new_j = -1; p.sem_slot = -1;
  p.fold_acc = nullptr; p.fold_logits = nullptr; p.fold_ml = nullptr;
  p.fold_pending = 0; p.fold_static = 0; p.fold_buffered = 0;
  p.early = (c->last_writer >= -1 && c->last_writer != layer) ? 1 : 0;
  p.scale_log2 = c->scale * 1.4426950408889634f;
  p.split = Split{0, 0, 0, 0, 0.f};
  c->fill_view(layer, p.view);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const bool timed = (size_t)(2 * c->prof_n + 1) < c->prof_ev.size();
  if (timed) cudaEventRecord(c->prof_ev[2 * c->prof_n], st);
  if ((c->kv_q8 ? launch_decode_q8(p, st) : launch_decode(p, st)) != cudaSuccess) return SSD_ERR_CUDA;
  c->last_writer = -1;
  if (c->row_buffer) {
    c->pending[layer] = 1;
    c->lg_cur[layer] = (uint8_t)lg_next;
  }
  if (timed) {
    cudaEventRecord(c->prof_ev[2 * c->prof_n + 1], st);
    c->prof_n += 1;
  }
  return SSD_OK;
}

int ssd_append_decode(ssd_cache* c, int32_t layer, const void* k_new, const void* v_new, const void* q, void* out,
                      void* stream) {
  if (!c || !k_new || !v_new || !q || !out) return SSD_ERR_INVALID_ARG;
  const ssd_config& g = c->cfg;
  if (layer < 0 || layer >= g.n_layers) return SSD_ERR_INVALID_ARG;
  if (!c->labels_set) return SSD_ERR_BAD_STATE;
  if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(out) | reinterpret_cast<uintptr_t>(k_new) |
       reinterpret_cast<uintptr_t>(v_new)) % 16 != 0)
    return SSD_ERR_INVALID_ARG;
  if (c->t_img[layer] >= g.max_image_tokens) return SSD_ERR_OVERFLOW;
  const bool scored = c->row_buffer && c->n_sink[layer] > 0;
  if (scored && c->sem_tokens(layer) >= g.sink_recent) return SSD_ERR_OVERFLOW;   // Algorithm 2, overflow branch
  DecodeParams p;
  p.slab = c->d_slab(layer);
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.out = static_cast<__nv_bfloat16*>(out);
  p.partial = c->d_partial();
  p.counters = c->d_counters();
  p.status = c->d_status();
  // Row-buffer mode (Algorithm 2): the launch records this step's logits in the layer's other buffer and,
  // at its start, adds the previous step's weights to the scores: still one launch
  const int lg_next = c->lg_cur[layer] ^ 1;
  p.logits = scored ? c->d_logits(layer, lg_next) : nullptr;
  p.ml = scored ? c->d_ml(layer, lg_next) : nullptr;
  p.mr = c->mr();
  p.sem_slot = scored ? c->sem_tokens(layer) : -1;
  p.fold_acc = scored ? c->d_acc(layer) : nullptr;
  p.fold_logits = c->d_logits(layer, c->lg_cur[layer]);
  p.fold_ml = c->d_ml(layer, c->lg_cur[layer]);
  p.fold_pending = scored && c->pending[layer] ? 1 : 0;
  p.fold_static = c->static_valid[layer];
  p.fold_buffered = c->sem_tokens(layer);
  p.k_new = static_cast<const unsigned char*>(k_new);
  p.v_new = static_cast<const unsigned char*>(v_new);
  p.new_j = c->t_img[layer];
  p.early = (c->last_writer >= -1 && c->last_writer != layer) ? 1 : 0;
  p.scale_log2 = c->scale * 1.4426950408889634f;
  p.split = Split{0, 0, 0, 0, 0.f};
  c->t_img[layer] += 1;                // the view describes the layer with the token in place
  c->fill_view(layer, p.view);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const bool timed = (size_t)(2 * c->prof_n + 1) < c->prof_ev.size();
  if (timed) cudaEventRecord(c->prof_ev[2 * c->prof_n], st);
  if ((c->kv_q8 ? launch_decode_q8(p, st) : launch_decode(p, st)) != cudaSuccess) {
    c->t_img[layer] -= 1;
    return SSD_ERR_CUDA;
  }
  c->last_writer = layer;
  if (scored) {
    c->pending[layer] = 1;
    c->lg_cur[layer] = (uint8_t)lg_next;
  }
  if (timed) {
    cudaEventRecord(c->prof_ev[2 * c->prof_n + 1], st);
    c->prof_n += 1;
  }
  return SSD_OK;
}

int ssd_append_decode_layers(ssd_cache* c, int32_t first_layer, int32_t n_layers, const void* k_new, const void* v_new,
                             const void* q, void* out, void* stream) {
  if (!c || !k_new || !v_new || !q || !out) return SSD_ERR_INVALID_ARG;
  const ssd_config& g = c->cfg;
  if (first_layer < 0 || n_layers < 1 || first_layer > g.n_layers - n_layers) return SSD_ERR_INVALID_ARG;
  if (n_layers > kMaxLayersPerLaunch) return SSD_ERR_LIMIT;
  if (!c->labels_set) return SSD_ERR_BAD_STATE;
  // Row buffer of one token: the launch re-selects as well (Algorithm 1 taken literally)
  const bool evict = c->row_buffer && g.sink_recent == 1;
  if (c->row_buffer && ((c->mr() + 3) & ~3) * (evict ? 3 : 1) > decode_layers_max_mr()) return SSD_ERR_LIMIT;
  if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(out) | reinterpret_cast<uintptr_t>(k_new) |
       reinterpret_cast<uintptr_t>(v_new)) % 16 != 0)
    return SSD_ERR_INVALID_ARG;
  for (int i = 0; i < n_layers; ++i) {
    const int layer = first_layer + i;
    if (c->t_img[layer] >= g.max_image_tokens) return SSD_ERR_OVERFLOW;
    if (c->row_buffer && c->n_sink[layer] > 0 && c->sem_tokens(layer) >= g.sink_recent)
      return SSD_ERR_OVERFLOW;          // Algorithm 2, overflow branch: call ssd_recompress first
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // Row-buffer mode: the kernel adds each step's attention weights to the scores itself.  A layer whose
  // last decode came from the per-layer call still has that step's weights pending: add them first.
  for (int i = 0; c->row_buffer && i < n_layers; ++i) {
    const int layer = first_layer + i;
    if (!c->pending[layer] || c->n_sink[layer] == 0) continue;
    if (launch_fold_pending(c->d_acc(layer), c->d_logits(layer, c->lg_cur[layer]), c->d_ml(layer, c->lg_cur[layer]),
                            c->d_desc(layer), g.n_seqs, g.n_heads,
                            c->mr(), c->static_valid[layer], c->sem_tokens(layer), st) != cudaSuccess)
      return SSD_ERR_CUDA;
    c->pending[layer] = 0;
  }
  DecodeLayersParams p = {};          // entries past n_layers stay zero
  p.slab = reinterpret_cast<uint4*>(c->base + c->reg.slab);
  p.q = static_cast<const unsigned char*>(q);
  p.k_new = static_cast<const unsigned char*>(k_new);
  p.v_new = static_cast<const unsigned char*>(v_new);
  p.out = static_cast<__nv_bfloat16*>(out);
  p.status = c->d_status();
  p.work = c->d_work();
  p.n_layers = n_layers; p.n_seqs = g.n_seqs; p.H = g.n_heads; p.L = g.prompt_len;
  p.acc = c->row_buffer ? c->d_acc(first_layer) : nullptr;
  p.static_idx = c->d_idx(first_layer);
  p.M = g.sink_budget;
  p.mr = c->row_buffer ? c->mr() : 0;
  p.evict = evict ? 1 : 0;
  p.scale_log2 = c->scale * 1.4426950408889634f;
  for (int i = 0; i < n_layers; ++i) {
    const int layer = first_layer + i;
    LayerState& ls = p.layer[i];
    ls.first_slot = c->layer_base[layer];
    ls.desc = c->d_desc(layer);
    ls.seq_slots = c->seq_slots[layer];
    ls.prompt_valid = c->prompt_valid[layer];
    ls.static_valid = c->static_valid[layer];
    ls.new_j = c->t_img[layer];
    ls.t_img = c->t_img[layer] + 1;
    ls.sem_slot = c->sem_tokens(layer);
    ls.t_sem = ls.sem_slot + 1;
  }
  if (cudaMemsetAsync(p.work, 0, 4, st) != cudaSuccess ||
      (c->kv_q8 ? launch_decode_layers_q8(p, st) : launch_decode_layers(p, st)) != cudaSuccess) {
    cudaGetLastError();
    return SSD_ERR_CUDA;
  }
  for (int i = 0; i < n_layers; ++i) {
    const int layer = first_layer + i;
    c->t_img[layer] += 1;
    c->pending[layer] = 0;             // this step's weights are already in the scores
    if (evict) {                       // and the buffer is empty again: the token entered the static set or left
      if (c->n_sink[layer] > 0 && c->static_valid[layer] < g.sink_budget) c->static_valid[layer] += 1;
      c->t_base[layer] = c->t_img[layer];
    }
  }
  c->last_writer = -2;                 // several layers' slabs were written
  return SSD_OK;
}

int ssd_step_host(ssd_cache* c, int32_t layer, const void* q_host, const void* k_new_host, const void* v_new_host,
                  void* out_host, void* stream) {
  if (!c || !q_host || !k_new_host || !v_new_host || !out_host) return SSD_ERR_INVALID_ARG;
  const ssd_config& g = c->cfg;
  if (layer < 0 || layer >= g.n_layers) return SSD_ERR_INVALID_ARG;
  if (!c->labels_set) return SSD_ERR_BAD_STATE;
  if (c->t_img[layer] >= g.max_image_tokens) return SSD_ERR_OVERFLOW;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t nb = (size_t)g.n_seqs * g.n_heads * kHeadDim * 2;
  char* s = c->d_staging();
  c->h_foreign = true;
  if (cudaMemcpyAsync(s, q_host, nb, cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemcpyAsync(s + nb, k_new_host, nb, cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemcpyAsync(s + 2 * nb, v_new_host, nb, cudaMemcpyHostToDevice, st) != cudaSuccess) {
    cudaGetLastError();
    return SSD_ERR_CUDA;
  }
  int rc = ssd_append_decode(c, layer, s + nb, s + 2 * nb, s, s + 3 * nb, stream);
  if (rc != SSD_OK) return rc;
  if (cudaMemcpyAsync(out_host, s + 3 * nb, nb, cudaMemcpyDeviceToHost, st) != cudaSuccess) {
    cudaGetLastError();
    return SSD_ERR_CUDA;
  }
  return SSD_OK;
}

int ssd_step_host_layers(ssd_cache* c, int32_t first_layer, int32_t n_layers, const void* q_host, const void* k_new_host,
                         const void* v_new_host, void* out_host, void* stream) {
  if (!c || !q_host || !k_new_host || !v_new_host || !out_host) return SSD_ERR_INVALID_ARG;
  const ssd_config& g = c->cfg;
  if (first_layer < 0 || n_layers < 1 || first_layer > g.n_layers - n_layers) return SSD_ERR_INVALID_ARG;
  if (!c->labels_set) return SSD_ERR_BAD_STATE;
  for (int i = 0; i < n_layers; ++i) {             // before anything is enqueued
    const int layer = first_layer + i;
    if (c->t_img[layer] >= g.max_image_tokens) return SSD_ERR_OVERFLOW;
    if (c->row_buffer && c->n_sink[layer] > 0 && c->sem_tokens(layer) >= g.sink_recent) return SSD_ERR_OVERFLOW;
  }
  if (!make_host_pipe(c)) return SSD_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t nb = (size_t)g.n_seqs * g.n_heads * kHeadDim * 2;
  const char* qh = static_cast<const char*>(q_host);
  const char* kh = static_cast<const char*>(k_new_host);
  const char* vh = static_cast<const char*>(v_new_host);
  char* oh = static_cast<char*>(out_host);
  bool ok = true;
  auto chk = [&](cudaError_t e) { ok = ok && e == cudaSuccess; };
  // The copies into a staging slot wait only for the kernels that last read that slot (events of the
  // ring, which carries on from call to call), not for the caller's stream as a whole: the next
  // step's inputs travel while this step's last kernels run.  If ssd_step_host has used the staging
  // area in between, the copy-in stream first waits for everything on the caller's stream.
  if (c->h_foreign) {
    chk(cudaEventRecord(c->h_fork, st));
    chk(cudaStreamWaitEvent(c->h_in, c->h_fork, 0));
    c->h_foreign = false;
  }
  int rc = SSD_OK;
  const size_t gb = (size_t)kHostGroup * nb;            // a slot is [q | k_new | v_new | out], each of a group
  for (int i0 = 0; ok && rc == SSD_OK && i0 < n_layers; i0 += kHostGroup) {
    const long grp = c->h_groups++;
    const int slot = (int)(grp % kHostSlots);
    const int cnt = n_layers - i0 < kHostGroup ? n_layers - i0 : kHostGroup;
    char* s = c->d_staging(slot);
    // inputs of a slot may be overwritten once the kernels that read them are done
    if (grp >= kHostSlots) chk(cudaStreamWaitEvent(c->h_in, c->h_done[slot], 0));
    chk(cudaMemcpyAsync(s, qh + (size_t)i0 * nb, cnt * nb, cudaMemcpyHostToDevice, c->h_in));
    chk(cudaMemcpyAsync(s + gb, kh + (size_t)i0 * nb, cnt * nb, cudaMemcpyHostToDevice, c->h_in));
    chk(cudaMemcpyAsync(s + 2 * gb, vh + (size_t)i0 * nb, cnt * nb, cudaMemcpyHostToDevice, c->h_in));
    chk(cudaEventRecord(c->h_loaded[slot], c->h_in));
    chk(cudaStreamWaitEvent(st, c->h_loaded[slot], 0));
    // the slot's outputs may be overwritten once its previous contents have gone to the host
    // (kHostSlots groups ago: long done, so this does not stall the kernels)
    if (grp >= kHostSlots) chk(cudaStreamWaitEvent(st, c->h_stored[slot], 0));
    if (!ok) break;
    for (int j = 0; j < cnt && rc == SSD_OK; ++j)
      rc = ssd_append_decode(c, first_layer + i0 + j, s + gb + j * nb, s + 2 * gb + j * nb, s + j * nb,
                             s + 3 * gb + j * nb, stream);
    if (rc != SSD_OK) break;
    chk(cudaEventRecord(c->h_done[slot], st));
    chk(cudaStreamWaitEvent(c->h_out, c->h_done[slot], 0));
    chk(cudaMemcpyAsync(oh + (size_t)i0 * nb, s + 3 * gb, cnt * nb, cudaMemcpyDeviceToHost, c->h_out));
    chk(cudaEventRecord(c->h_stored[slot], c->h_out));
  }
  // join: the caller's stream is not done before the outputs are on the host (the kernels have
  // already waited for the inputs)
  for (int slot = 0; slot < kHostSlots; ++slot) cudaStreamWaitEvent(st, c->h_stored[slot], 0);
  if (rc != SSD_OK) return rc;
  if (!ok) {
    cudaGetLastError();
    return SSD_ERR_CUDA;
  }
  return SSD_OK;
}

int32_t ssd_cache_max_slots(const ssd_cache* c) { return c ? c->max_slots() : -1; }

int ssd_cache_get_indices(ssd_cache* c, int32_t layer, int32_t* idx_host) {
  if (!c || !idx_host) return SSD_ERR_INVALID_ARG;
  const ssd_config& g = c->cfg;
  if (layer < 0 || layer >= g.n_layers) return SSD_ERR_INVALID_ARG;
  if (!c->labels_set) return SSD_ERR_BAD_STATE;
  const int ms = c->max_slots(), M = g.sink_budget;
  std::vector<int32_t> sidx((size_t)g.n_seqs * g.n_heads * (M > 0 ? M : 1));
  if (cudaDeviceSynchronize() != cudaSuccess ||
      cudaMemcpy(sidx.data(), c->d_idx(layer), sidx.size() * 4, cudaMemcpyDeviceToHost) != cudaSuccess) {
    cudaGetLastError();
    return SSD_ERR_CUDA;
  }
  const int t = c->t_img[layer], L = g.prompt_len;
  for (int s = 0; s < g.n_seqs; ++s)
    for (int h = 0; h < g.n_heads; ++h) {
      const HeadDesc& d = c->desc[(size_t)layer * g.n_heads + h];
      int32_t* o = idx_host + ((size_t)s * g.n_heads + h) * ms;
      for (int i = 0; i < ms; ++i) o[i] = -1;
      for (int i = 0; i < c->prompt_valid[layer]; ++i) o[i] = i;
      if (d.w)
        for (int m = 0; m < c->static_valid[layer]; ++m) {
          int j = sidx[((size_t)s * g.n_heads + h) * (M > 0 ? M : 1) + m];
          o[L + m] = j >= 0 ? L + j : -1;
        }
      if (d.w && c->row_buffer) {       // row buffer: filled from slot 0 since the last re-selection
        for (int r = 0; r < c->sem_tokens(layer) && r < d.z; ++r) o[L + d.y + r] = L + c->t_base[layer] + r;
      } else {
        for (int r = 0; r < d.z; ++r)
          if (t - 1 >= r) o[L + d.y + r] = L + ((t - 1 - r) / d.z) * d.z + r;
      }
    }
  return SSD_OK;
}

int ssd_cache_get_lengths(ssd_cache* c, int32_t layer, int32_t* len_host) {
  if (!c || !len_host) return SSD_ERR_INVALID_ARG;
  const ssd_config& g = c->cfg;
  if (layer < 0 || layer >= g.n_layers) return SSD_ERR_INVALID_ARG;
  if (!c->labels_set) return SSD_ERR_BAD_STATE;
  for (int h = 0; h < g.n_heads; ++h) {
    const HeadDesc& d = c->desc[(size_t)layer * g.n_heads + h];
    const int tok = d.w ? c->sem_tokens(layer) : c->t_img[layer];
    len_host[h] = c->prompt_valid[layer] + (d.w ? c->static_valid[layer] : 0) + (tok < d.z ? tok : d.z);
  }
  return SSD_OK;
}

int ssd_cache_get_labels(ssd_cache* c, uint8_t* labels_host) {
  if (!c || !labels_host) return SSD_ERR_INVALID_ARG;
  if (!c->labels_set) return SSD_ERR_BAD_STATE;
  std::memcpy(labels_host, c->labels.data(), c->labels.size());
  return SSD_OK;
}

int32_t ssd_cache_tokens(const ssd_cache* c, int32_t layer) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers) return -1;
  return c->t_img[layer];
}

int ssd_cache_rewind(ssd_cache* c, int32_t layer, int32_t t) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers) return SSD_ERR_INVALID_ARG;
  if (t < c->n0[layer] || t > c->t_img[layer]) return SSD_ERR_INVALID_ARG;
  if (c->row_buffer) return SSD_ERR_BAD_STATE;   // the static sets have moved on; replay is meaningless
  c->t_img[layer] = t;
  return SSD_OK;
}

int ssd_cache_kv_bytes(ssd_cache* c, size_t* bytes_per_seq) {
  if (!c || !bytes_per_seq) return SSD_ERR_INVALID_ARG;
  if (!c->labels_set) return SSD_ERR_BAD_STATE;
  size_t slots = 0;
  for (int l = 0; l < c->cfg.n_layers; ++l) slots += (size_t)c->seq_slots[l];
  *bytes_per_seq = slots * (size_t)c->slot_bytes();
  return SSD_OK;
}

int ssd_cache_set_kv_format(ssd_cache* c, int32_t format) {
  if (!c || (format != 0 && format != 1)) return SSD_ERR_INVALID_ARG;
  if (format == 1 && c->row_buffer) return SSD_ERR_BAD_STATE;
  c->kv_q8 = format == 1;
  for (int l = 0; l < c->cfg.n_layers; ++l) {
    c->t_img[l] = c->n0[l] = c->prompt_valid[l] = c->static_valid[l] = c->t_base[l] = 0;
    c->pending[l] = 0;
  }
  return SSD_OK;
}

int ssd_quantize_rows_e4m3(const void* rows, int64_t n_rows, void* codes_out, float* scales_out, void* stream) {
  if (!rows || !codes_out || !scales_out || n_rows < 0 || n_rows > (int64_t)1 << 36) return SSD_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(rows) | reinterpret_cast<uintptr_t>(codes_out)) % 16 != 0 ||
      reinterpret_cast<uintptr_t>(scales_out) % 4 != 0)
    return SSD_ERR_INVALID_ARG;
  if (n_rows == 0) return SSD_OK;
  return launch_quantize_rows(rows, n_rows, codes_out, scales_out, static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? SSD_OK : SSD_ERR_CUDA;
}

int ssd_cache_set_row_buffer(ssd_cache* c, int32_t enable) {
  if (!c) return SSD_ERR_INVALID_ARG;
  if (enable && c->kv_q8) return SSD_ERR_BAD_STATE;
  c->row_buffer = enable != 0;
  for (int l = 0; l < c->cfg.n_layers; ++l) {
    c->t_img[l] = c->n0[l] = c->prompt_valid[l] = c->static_valid[l] = c->t_base[l] = 0;
    c->pending[l] = 0;
  }
  return SSD_OK;
}

int ssd_recompress(ssd_cache* c, int32_t layer, void* stream) {
  if (!c) return SSD_ERR_INVALID_ARG;
  const ssd_config& g = c->cfg;
  if (layer < 0 || layer >= g.n_layers) return SSD_ERR_INVALID_ARG;
  if (!c->labels_set || !c->row_buffer) return SSD_ERR_BAD_STATE;
  const int buffered = c->sem_tokens(layer);
  if (c->n_sink[layer] > 0 && (buffered > 0 || c->pending[layer])) {
    RecompressParams p;
    p.slab = c->d_slab(layer);
    p.desc = c->d_desc(layer);
    p.static_idx = c->d_idx(layer);
    p.acc = c->d_acc(layer);
    p.logits = c->d_logits(layer, c->lg_cur[layer]);
    p.ml = c->d_ml(layer, c->lg_cur[layer]);
    p.pending = c->pending[layer];
    p.n_seqs = g.n_seqs; p.H = g.n_heads; p.L = g.prompt_len; p.M = g.sink_budget; p.mr = c->mr();
    p.static_valid = c->static_valid[layer];
    p.buffered = buffered;
    p.t_base = c->t_base[layer];
    p.seq_slots = c->seq_slots[layer];
    if (launch_recompress(p, static_cast<cudaStream_t>(stream)) != cudaSuccess) return SSD_ERR_CUDA;
    const int n = c->static_valid[layer] + buffered;
    c->static_valid[layer] = n < g.sink_budget ? n : g.sink_budget;
  }
  c->t_base[layer] = c->t_img[layer];
  c->pending[layer] = 0;
  c->last_writer = -2;
  return SSD_OK;
}

int ssd_recompress_layers(ssd_cache* c, int32_t first_layer, int32_t n_layers, void* stream) {
  if (!c) return SSD_ERR_INVALID_ARG;
  const ssd_config& g = c->cfg;
  if (first_layer < 0 || n_layers < 1 || first_layer > g.n_layers - n_layers) return SSD_ERR_INVALID_ARG;
  if (n_layers > kMaxLayersPerLaunch) return SSD_ERR_LIMIT;
  if (!c->labels_set || !c->row_buffer) return SSD_ERR_BAD_STATE;
  RecompressLayersParams p = {};      // entries past n_layers stay zero
  p.slab = reinterpret_cast<uint4*>(c->base + c->reg.slab);
  p.desc = c->d_desc(first_layer);
  p.static_idx = c->d_idx(first_layer);
  p.acc = c->d_acc(first_layer);
  p.logits = c->d_logits(first_layer, 0);
  p.ml = c->d_ml(first_layer, 0);
  p.n_layers = n_layers; p.n_seqs = g.n_seqs; p.H = g.n_heads; p.L = g.prompt_len; p.M = g.sink_budget; p.mr = c->mr();
  bool any = false;
  for (int i = 0; i < n_layers; ++i) {
    const int layer = first_layer + i;
    RecompressLayer& ly = p.layer[i];
    ly.first_slot = c->layer_base[layer];
    ly.seq_slots = c->seq_slots[layer];
    ly.static_valid = c->static_valid[layer];
    ly.buffered = c->sem_tokens(layer);
    ly.t_base = c->t_base[layer];
    ly.pending = c->pending[layer];
    ly.lg = c->lg_cur[layer];
    ly.todo = (c->n_sink[layer] > 0 && (ly.buffered > 0 || ly.pending)) ? 1 : 0;
    any = any || ly.todo;
  }
  // a buffer of one token (Algorithm 1 taken literally) needs no ranking: drop the lowest score
  if (any && (g.sink_recent == 1 ? launch_evict_one_layers(p, static_cast<cudaStream_t>(stream))
                                 : launch_recompress_layers(p, static_cast<cudaStream_t>(stream))) != cudaSuccess)
    return SSD_ERR_CUDA;
  for (int i = 0; i < n_layers; ++i) {
    const int layer = first_layer + i;
    if (p.layer[i].todo) {
      const int n = c->static_valid[layer] + p.layer[i].buffered;
      c->static_valid[layer] = n < g.sink_budget ? n : g.sink_budget;
    }
    c->t_base[layer] = c->t_img[layer];
    c->pending[layer] = 0;
  }
  c->last_writer = -2;
  return SSD_OK;
}

int ssd_cache_get_scores(ssd_cache* c, int32_t layer, float* acc_host) {
  if (!c || !acc_host) return SSD_ERR_INVALID_ARG;
  const ssd_config& g = c->cfg;
  if (layer < 0 || layer >= g.n_layers) return SSD_ERR_INVALID_ARG;
  if (!c->labels_set || !c->row_buffer) return SSD_ERR_BAD_STATE;
  const size_t n = (size_t)g.n_seqs * g.n_heads * c->mr();
  std::vector<float> lg(n);
  std::vector<float2> ml((size_t)g.n_seqs * g.n_heads);
  if (cudaDeviceSynchronize() != cudaSuccess ||
      cudaMemcpy(acc_host, c->d_acc(layer), n * 4, cudaMemcpyDeviceToHost) != cudaSuccess ||
      cudaMemcpy(lg.data(), c->d_logits(layer, c->lg_cur[layer]), n * 4, cudaMemcpyDeviceToHost) != cudaSuccess ||
      cudaMemcpy(ml.data(), c->d_ml(layer, c->lg_cur[layer]), ml.size() * 8, cudaMemcpyDeviceToHost) != cudaSuccess) {
    cudaGetLastError();
    return SSD_ERR_CUDA;
  }
  const int mr = c->mr(), sv = c->static_valid[layer], b = c->sem_tokens(layer);
  for (int pr = 0; pr < g.n_seqs * g.n_heads; ++pr) {
    const HeadDesc& d = c->desc[(size_t)layer * g.n_heads + pr % g.n_heads];
    float* a = acc_host + (size_t)pr * mr;
    for (int e = 0; e < mr; ++e) {
      const bool valid = d.w && (e < sv || (e >= d.y && e < d.y + b));
      if (!valid) { a[e] = -1.f; continue; }
      // what the next append or re-selection would add first: the last decode's normalised weights
      if (c->pending[layer]) a[e] += std::exp2(lg[(size_t)pr * mr + e] - ml[pr].x) / ml[pr].y;
    }
  }
  return SSD_OK;
}

int ssd_cache_get_compress_scores(ssd_cache* c, int32_t layer, float* score_host) {
  if (!c || !score_host) return SSD_ERR_INVALID_ARG;
  const ssd_config& g = c->cfg;
  if (layer < 0 || layer >= g.n_layers) return SSD_ERR_INVALID_ARG;
  if (c->score_layer != layer || c->score_n0 < 1) return SSD_ERR_BAD_STATE;
  // a pair's score row is the first of its kScoreHalves rows (the selection has added the others into it)
  if (cudaDeviceSynchronize() != cudaSuccess ||
      cudaMemcpy2D(score_host, (size_t)c->score_n0 * 4, c->d_score(), (size_t)kScoreHalves * c->score_n0 * 4,
                   (size_t)c->score_n0 * 4, (size_t)g.n_seqs * g.n_heads, cudaMemcpyDeviceToHost) != cudaSuccess) {
    cudaGetLastError();
    return SSD_ERR_CUDA;
  }
  for (int pr = 0; pr < g.n_seqs * g.n_heads; ++pr)
    if (!c->desc[(size_t)layer * g.n_heads + pr % g.n_heads].w)
      for (int j = 0; j < c->score_n0; ++j) score_host[(size_t)pr * c->score_n0 + j] = -1.f;
  return SSD_OK;
}

int ssd_cache_device_status(ssd_cache* c, uint32_t* status_host) {
  if (!c || !status_host) return SSD_ERR_INVALID_ARG;
  if (cudaDeviceSynchronize() != cudaSuccess ||
      cudaMemcpy(status_host, c->d_status(), 4, cudaMemcpyDeviceToHost) != cudaSuccess) {
    cudaGetLastError();
    return SSD_ERR_CUDA;
  }
  return SSD_OK;
}

int64_t ssd_debug_decode_plan(int32_t n_heads, const int32_t* head_recs, int32_t prompt_len, int32_t n_seqs,
                              int32_t prompt_valid, int32_t static_valid, int32_t t_img, int32_t max_workers,
                              int32_t chunk, int64_t* copies_out, int64_t cap) {
  if (n_heads < 1 || n_heads > kMaxHeads || !head_recs || n_seqs < 1 || prompt_len < 0 || max_workers < 1)
    return SSD_ERR_INVALID_ARG;
  if ((prompt_valid != 0 && prompt_valid != prompt_len) || static_valid < 0 || t_img < 0 || cap < 0 ||
      (cap > 0 && !copies_out))
    return SSD_ERR_INVALID_ARG;
  if (chunk <= 0) chunk = decode_chunk_slots();
  LayerView v;
  v.H = n_heads; v.L = prompt_len; v.n_seqs = n_seqs;
  v.prompt_valid = prompt_valid; v.static_valid = static_valid; v.t_img = t_img; v.t_sem = t_img;
  int off = 0;
  for (int h = 0; h < n_heads; ++h) {
    const int32_t* r = head_recs + 4 * h;
    if (r[1] < 0 || r[2] < 1 || r[0] != off || (r[3] == 0 && r[1] != 0) || (r[3] != 0 && static_valid > r[1]))
      return SSD_ERR_INVALID_ARG;
    v.head[h] = HeadRec{r[0], r[1], r[2], r[3]};
    off += prompt_len + r[1] + r[2];
  }
  v.seq_slots = off;
  view_finish(v);
  const int run = v.cum[n_heads];
  const long T = (long)run * n_seqs;
  if (T < 1) return SSD_ERR_BAD_STATE;
  if (T > 0x7fffffffL) return SSD_ERR_INVALID_ARG;
  const long W = plan_workers(T, max_workers);
  const Split sp = make_split(T, W);
  int64_t n = 0;
  for (int32_t wk = 0; wk < (int32_t)W; ++wk) {
    const Share sh = share_plan(v, sp, wk);
    if (sh.g_begin >= sh.g_end) continue;
    if (share_of(sp, sh.g_begin) != wk || share_of(sp, sh.g_end - 1) != wk) return SSD_ERR_BAD_STATE;
    Walk w;
    walk_init(w, v, sh.g_begin, sh.g_end);
    int64_t k = 0;
    while (w.g < w.g_end) {
      const int nn = walk_chunk(w, chunk);
      if (nn < 1) return SSD_ERR_BAD_STATE;
      const int64_t hbase = (int64_t)w.seq * v.seq_slots + v.head[w.head].x;
      auto emit = [&](int src, int dst, int len) {
        if (n < cap) {
          int64_t* o = copies_out + 6 * n;
          o[0] = wk; o[1] = k; o[2] = hbase + src; o[3] = dst; o[4] = len; o[5] = (int64_t)w.seq * n_heads + w.head;
        }
        ++n;
      };
      if (v.contig) emit(w.i, 0, nn);   // the kernel's fast path: one copy per chunk
      else chunk_runs(v, w.head, w.i, nn, emit);
      walk_advance(w, v, nn);
      ++k;
    }
  }
  return n;
}

}  // extern "C"

// ------------------------------------------------------------------------------------------------
// Decode attention for callers that cannot hand the library any scratch memory of their own.
// The cross-block partials and the per-head arrival counters of the decode kernel live in this
// array, which is part of the library image: every GPU that loads the library carries it until
// the process exits.  Layout: [kStaticCtas * 2 partials of kPartialFloats floats | kStaticPairs
// counters].
namespace {
constexpr int kStaticCtas = 256;       // thread blocks (one per SM) the partial area has room for
constexpr int kStaticPairs = 32768;    // (sequence, head) pairs the counter area has room for
constexpr size_t kStaticPartialBytes = (size_t)kStaticCtas * 2 * ssd::kPartialFloats * 4;
constexpr size_t kStaticBytes = kStaticPartialBytes + (size_t)kStaticPairs * 4;
}  // namespace

static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

extern "C" int ssd_decode_attn_static(ssd_cache* c, int32_t layer, const void* q, void* out, void* stream) {
  if (!c || !q || !out) return SSD_ERR_INVALID_ARG;
  const ssd_config& g = c->cfg;
  if (layer < 0 || layer >= g.n_layers) return SSD_ERR_INVALID_ARG;
  if (!c->labels_set || c->kv_q8) return SSD_ERR_BAD_STATE;
  if (c->empty_head(layer, c->t_img[layer], c->sem_tokens(layer))) return SSD_ERR_BAD_STATE;
  if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(out)) % 16 != 0) return SSD_ERR_INVALID_ARG;
  const long pairs = (long)g.n_seqs * g.n_heads;
  if (pairs > kStaticPairs) return SSD_ERR_LIMIT;

  // Once per device, with that device current: the array's name is only a host-side handle here,
  // so ask the runtime where the array lives on this device.
  // (two host threads that make their first call at once both look the address up and store the same value)
  static std::atomic<unsigned char*> dev_ptr[64] = {};
  static std::atomic<int> dev_sms[64] = {};
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
    cudaGetLastError();
    return SSD_ERR_CUDA;
  }
  unsigned char* base = dev_ptr[dev].load(std::memory_order_acquire);
  if (!base) {
    void* ptr = nullptr;
    int sms = 0;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
      cudaGetLastError();
      return SSD_ERR_CUDA;
    }
    dev_sms[dev].store(sms, std::memory_order_relaxed);
    base = static_cast<unsigned char*>(ptr);
    dev_ptr[dev].store(base, std::memory_order_release);
  }
  if (dev_sms[dev].load(std::memory_order_relaxed) > kStaticCtas) return SSD_ERR_LIMIT;   // the kernel runs one thread block per SM

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // The array keeps what the previous call left.  Partials are written before they are read, but
  // the arrival counters must start at zero, which a call that was cut short would not guarantee.
  if (cudaMemsetAsync(base + kStaticPartialBytes, 0, (size_t)pairs * 4, st) != cudaSuccess) {
    cudaGetLastError();
    return SSD_ERR_CUDA;
  }
  DecodeParams p;
  p.slab = c->d_slab(layer);
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.out = static_cast<__nv_bfloat16*>(out);
  p.partial = reinterpret_cast<float*>(base);
  p.counters = reinterpret_cast<uint32_t*>(base + kStaticPartialBytes);
  p.status = c->d_status();
  const int lg_next = c->lg_cur[layer] ^ 1;
  p.logits = c->row_buffer ? c->d_logits(layer, lg_next) : nullptr;
  p.ml = c->row_buffer ? c->d_ml(layer, lg_next) : nullptr;
  p.mr = c->mr();
  p.k_new = nullptr; p.v_new = nullptr; p.new_j = -1; p.sem_slot = -1;
  p.fold_acc = nullptr; p.fold_logits = nullptr; p.fold_ml = nullptr;
  p.fold_pending = 0; p.fold_static = 0; p.fold_buffered = 0;
  p.early = (c->last_writer >= -1 && c->last_writer != layer) ? 1 : 0;
  p.scale_log2 = c->scale * 1.4426950408889634f;
  p.split = Split{0, 0, 0, 0, 0.f};
  c->fill_view(layer, p.view);
  if (launch_decode(p, st) != cudaSuccess) return SSD_ERR_CUDA;
  c->last_writer = -1;
  if (c->row_buffer) {
    c->pending[layer] = 1;
    c->lg_cur[layer] = (uint8_t)lg_next;
  }
  return SSD_OK;
}
