// Host side of the C ABI: argument validation, the pyramid schedule
// (Algorithm 1: ratio p per layer, minimum PvC lengths N_l), carving of the
// caller's device buffer, call ordering, and dispatch to the kernels.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstring>
#include <new>
#include <vector>

#include "pyr_internal.h"

namespace {

struct LayerPlan {
  int n_in, c, k, n_out, cap;
  size_t k_off, v_off;   // byte offsets into the device buffer
  size_t q_off;          // ring of recent queries (generation-phase re-selection only)
};

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

constexpr size_t kAlign = 256;

std::atomic<uint64_t> g_launches{0};   // kernels launched by this process through the library
std::atomic<int> g_sm_count[64];        // per device, 0 = not asked yet

struct Layout {
  size_t status, w, score, score_part, lse, idx, rank, pos0, pos1, part_acc, part_ml, gen_part, total;
  int q_ring;            // rows of a layer's query ring (0: no generation-phase re-selection)
  std::vector<LayerPlan> layers;
};

pyr_status_t validate(const pyr_config_t* c) {
  if (!c) return PYR_ERR_NULL;
  if (!c->ratio) return PYR_ERR_NULL;
  if (c->n_layers < 1 || c->n_q_heads < 1 || c->n_kv_heads < 1 || c->batch < 1 ||
      c->prompt_len < 1 || c->recent_len < 1 || c->max_new_tokens < 0)
    return PYR_ERR_INVALID;
  if (c->n_q_heads % c->n_kv_heads != 0) return PYR_ERR_INVALID;
  if (c->sel_groups != 1 && c->sel_groups != c->n_kv_heads) return PYR_ERR_INVALID;
  if (c->dtype != PYR_BF16 && c->dtype != PYR_F32) return PYR_ERR_UNSUPPORTED;
  if (c->head_dim != 64 && c->head_dim != 128) return PYR_ERR_UNSUPPORTED;
  if (c->prompt_len > pyr::kMaxPrompt) return PYR_ERR_UNSUPPORTED;
  if (!(c->softmax_scale >= 0.0f) || !std::isfinite(c->softmax_scale)) return PYR_ERR_INVALID;
  double prev = 1.0;
  for (int l = 0; l < c->n_layers; ++l) {
    double r = c->ratio[l];
    if (!(r >= 0.0 && r <= 1.0)) return PYR_ERR_INVALID;
    if (r > prev) return PYR_ERR_INVALID;
    prev = r;
    if (c->min_len && c->min_len[l] < 0) return PYR_ERR_INVALID;
  }
  if (c->recent_w) {
    int L = c->recent_len;
    for (int i = 0; i < L; ++i)
      if (!(c->recent_w[i] >= 0.0f) || !std::isfinite(c->recent_w[i])) return PYR_ERR_INVALID;
  }
  return PYR_OK;
}

// Budgets: k_l = min(c, max(floor(ratio_l * c_0), N_l - L, 0)); the window is
// never evicted; a layer with no context keeps everything.
void plan(const pyr_config_t* c, Layout* lay) {
  const int N = c->prompt_len, L = c->recent_len;
  const int c0 = N > L ? N - L : 0;
  const size_t eb = c->dtype == PYR_BF16 ? 2 : 4;
  const size_t B = c->batch, G = c->sel_groups, Hq = c->n_q_heads, Hkv = c->n_kv_heads,
               D = c->head_dim;
  size_t off = 0;
  lay->status = off; off = align_up(off + pyr::kStatusWords * sizeof(int), kAlign);
  lay->w = off;      off = align_up(off + (size_t)L * 4, kAlign);
  const bool gen = (c->flags & PYR_FLAG_GEN_RESELECT) != 0;
  // generation-phase re-selection scores up to c_0 + T context rows (the kept context plus the decode rows)
  const size_t c_max = (size_t)(c0 > 0 ? c0 : 1) + (gen ? (size_t)c->max_new_tokens : 0);
  lay->score = off;  off = align_up(off + B * G * c_max * 4, kAlign);
  // per-head partial scores of the tensor-core score kernel (bf16, head_dim 128 only)
  lay->score_part = off;
  if (c->dtype == PYR_BF16 && D == 128 && c0 > 0)
    off = align_up(off + B * Hq * (size_t)pyr::score_tc_chunks(L) * pyr::score_tc_groups() * (size_t)c0 * 4, kAlign);
  lay->lse = off;    off = align_up(off + B * Hq * (size_t)N * 4, kAlign);
  lay->idx = off;    off = align_up(off + B * G * (size_t)N * 4, kAlign);
  lay->rank = off;
  if (c->flags & PYR_FLAG_SELECT_FIRST) off = align_up(off + B * G * (size_t)N * 4, kAlign);   // the inverse of idx
  lay->pos0 = off;   off = align_up(off + B * G * (size_t)N * 4, kAlign);
  lay->pos1 = off;   off = align_up(off + B * G * (size_t)N * 4, kAlign);
  lay->part_acc = off;
  if (c->max_new_tokens > 0) off = align_up(off + B * Hq * pyr::kMaxDecodeSplits * D * 4, kAlign);
  lay->part_ml = off;
  if (c->max_new_tokens > 0) off = align_up(off + B * Hq * pyr::kMaxDecodeSplits * 2 * 4, kAlign);
  lay->gen_part = off;
  if (gen) off = align_up(off + B * Hq * (size_t)pyr::gen_score_qtiles(L) * c_max * 4, kAlign);
  lay->q_ring = gen ? L + (c->max_new_tokens > 0 ? c->max_new_tokens : 1) : 0;
  lay->layers.resize(c->n_layers);
  int n_in = N;
  for (int l = 0; l < c->n_layers; ++l) {
    LayerPlan& p = lay->layers[l];
    p.n_in = n_in;
    p.c = n_in > L ? n_in - L : 0;
    const int window = n_in - p.c;
    long long want = (long long)std::floor(c->ratio[l] * (double)c0);
    long long lo = c->min_len ? (long long)c->min_len[l] - L : 0;
    long long k = want > lo ? want : lo;
    if (k < 0) k = 0;
    if (k > p.c) k = p.c;
    p.k = (int)k;
    p.n_out = p.k + window;
    p.cap = p.n_out + c->max_new_tokens;
    const size_t bytes = B * Hkv * (size_t)p.cap * D * eb;
    p.k_off = off; off = align_up(off + bytes, kAlign);
    p.v_off = off; off = align_up(off + bytes, kAlign);
    p.q_off = off;
    if (gen) off = align_up(off + B * (size_t)lay->q_ring * Hq * D * eb, kAlign);
    n_in = p.n_out;
  }
  lay->total = off;
}

}  // namespace

namespace pyr {

int device_sm_count() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
  int n = g_sm_count[dev].load();
  if (n == 0) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 0;
    g_sm_count[dev].store(n);
  }
  return n;
}

void count_launches(int kernels) { g_launches += (uint64_t)kernels; }

}  // namespace pyr

struct pyr_cache {
  pyr_config_t cfg;
  std::vector<double> ratio;
  std::vector<int32_t> min_len;
  std::vector<float> w;
  Layout lay;
  char* base;
  std::vector<int> len_now;
  std::vector<long long> q_count;   // queries written to each layer's ring so far
  int next_layer;     // layer whose prefill (phase 0) or select (phase 1) comes next
  int phase;
  int pos_cur;        // which of pos0/pos1 holds the positions of the last selection
  int last_selected;  // layer of the last pyr_select_compact, -1 if none
  int last_prefilled;
  bool needs_init;
  bool wait_test_armed;   // pyr_cache_arm_wait_test: the next decode call's loader leaves a chunk out
  const void* sf_out;     // select-first ordering: the output tensor whose rows the last prefill wrote in kept order
                          // (null: the selection has not run yet)
  int sf_boundary;        // first row of the query tiles that were written before the selection
  float scale;
};

namespace {

template <class T>
T* at(const pyr_cache* c, size_t off) { return reinterpret_cast<T*>(c->base + off); }

pyr_status_t device_init(pyr_cache* c, cudaStream_t s) {
  if (cudaMemsetAsync(at<int>(c, c->lay.status), 0, pyr::kStatusWords * sizeof(int), s) != cudaSuccess)
    return PYR_ERR_CUDA;
  if (c->needs_init) {
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return PYR_ERR_CUDA;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
      return PYR_ERR_CUDA;
    if (major != 10) return PYR_ERR_UNSUPPORTED;
    if (cudaMemcpyAsync(at<float>(c, c->lay.w), c->w.data(), c->w.size() * 4, cudaMemcpyHostToDevice,
                        s) != cudaSuccess)
      return PYR_ERR_CUDA;
    c->needs_init = false;
  }
  return PYR_OK;
}

}  // namespace

extern "C" {

const char* pyr_status_string(pyr_status_t s) {
  switch (s) {
    case PYR_OK: return "ok";
    case PYR_ERR_INVALID: return "invalid argument";
    case PYR_ERR_NULL: return "null pointer";
    case PYR_ERR_UNSUPPORTED: return "unsupported dtype, head_dim, size or device";
    case PYR_ERR_BUFFER_TOO_SMALL: return "device buffer too small";
    case PYR_ERR_CAPACITY: return "layer cache is full";
    case PYR_ERR_ORDER: return "call out of sequence";
    case PYR_ERR_CUDA: return "CUDA runtime error";
    case PYR_ERR_TIMEOUT: return "device-side wait timed out";
    case PYR_ERR_SCRATCH_LIMIT: return "problem needs more scratch than the library's built-in array holds";
    case PYR_ERR_HOST_MEMORY: return "out of host memory";
  }
  return "unknown status";
}

int32_t pyr_version(void) { return 100; }

uint64_t pyr_launch_count(void) { return g_launches.load(); }

pyr_status_t pyr_cache_bytes(const pyr_config_t* cfg, size_t* bytes, size_t* align) {
  pyr_status_t st = validate(cfg);
  if (st != PYR_OK) return st;
  if (!bytes) return PYR_ERR_NULL;
  try {
    Layout lay;
    plan(cfg, &lay);
    *bytes = lay.total;
  } catch (...) {
    return PYR_ERR_HOST_MEMORY;
  }
  if (align) *align = kAlign;
  return PYR_OK;
}

pyr_status_t pyr_cache_alloc(const pyr_config_t* cfg, void* dev_buf, size_t bytes, pyr_cache_t** out) {
  pyr_status_t st = validate(cfg);
  if (st != PYR_OK) return st;
  if (!dev_buf || !out) return PYR_ERR_NULL;
  if (reinterpret_cast<uintptr_t>(dev_buf) % kAlign) return PYR_ERR_INVALID;
  pyr_cache* c = new (std::nothrow) pyr_cache();
  if (!c) return PYR_ERR_HOST_MEMORY;
  try {
  c->cfg = *cfg;
  c->ratio.assign(cfg->ratio, cfg->ratio + cfg->n_layers);
  if (cfg->min_len) c->min_len.assign(cfg->min_len, cfg->min_len + cfg->n_layers);
  c->cfg.ratio = c->ratio.data();
  c->cfg.min_len = cfg->min_len ? c->min_len.data() : nullptr;
  const int L = cfg->recent_len;
  c->w.resize(L);
  for (int i = 0; i < L; ++i)
    c->w[i] = cfg->recent_w ? cfg->recent_w[i]
                            : (float)(2.0 * (i + 1.0) / ((double)L * (double)(L + 1)));
  c->cfg.recent_w = c->w.data();
  plan(&c->cfg, &c->lay);
  if (bytes < c->lay.total) { delete c; return PYR_ERR_BUFFER_TOO_SMALL; }
  c->base = static_cast<char*>(dev_buf);
  c->len_now.assign(cfg->n_layers, 0);
  c->q_count.assign(cfg->n_layers, 0);
  c->next_layer = 0; c->phase = 0; c->pos_cur = 0; c->last_selected = -1; c->last_prefilled = -1;
  c->needs_init = true;
  c->wait_test_armed = false;
  c->sf_out = nullptr; c->sf_boundary = 0;
  c->scale = cfg->softmax_scale > 0.0f ? cfg->softmax_scale : (float)(1.0 / std::sqrt((double)cfg->head_dim));
  } catch (...) {           // the host-side vectors could not be allocated
    delete c;
    return PYR_ERR_HOST_MEMORY;
  }
  *out = c;
  return PYR_OK;
}

pyr_status_t pyr_cache_free(pyr_cache_t* c) {
  if (!c) return PYR_ERR_NULL;
  delete c;
  return PYR_OK;
}

pyr_status_t pyr_cache_reset(pyr_cache_t* c, void* stream) {
  if (!c) return PYR_ERR_NULL;
  c->next_layer = 0; c->phase = 0; c->pos_cur = 0; c->last_selected = -1; c->last_prefilled = -1;
  c->sf_out = nullptr;
  std::fill(c->len_now.begin(), c->len_now.end(), 0);
  std::fill(c->q_count.begin(), c->q_count.end(), 0);
  return device_init(c, static_cast<cudaStream_t>(stream));
}

pyr_status_t pyr_cache_layer_info(const pyr_cache_t* c, int32_t layer, int32_t* n_in, int32_t* k_ctx,
                                  int32_t* len_now, int32_t* cap) {
  if (!c) return PYR_ERR_NULL;
  if (layer < 0 || layer >= c->cfg.n_layers) return PYR_ERR_INVALID;
  const LayerPlan& p = c->lay.layers[layer];
  if (n_in) *n_in = p.n_in;
  if (k_ctx) *k_ctx = p.k;
  if (len_now) *len_now = c->len_now[layer];
  if (cap) *cap = p.cap;
  return PYR_OK;
}

pyr_status_t pyr_cache_kept(const pyr_cache_t* c, int32_t layer, const int32_t** dev_idx,
                            const int32_t** dev_pos) {
  if (!c) return PYR_ERR_NULL;
  if (layer < 0 || layer >= c->cfg.n_layers) return PYR_ERR_INVALID;
  if (layer != c->last_selected) return PYR_ERR_ORDER;
  if (dev_idx) *dev_idx = at<int32_t>(c, c->lay.idx);
  if (dev_pos) *dev_pos = at<int32_t>(c, c->pos_cur ? c->lay.pos1 : c->lay.pos0);
  return PYR_OK;
}

pyr_status_t pyr_cache_scores(const pyr_cache_t* c, int32_t layer, const float** dev_scores) {
  if (!c || !dev_scores) return PYR_ERR_NULL;
  if (layer < 0 || layer >= c->cfg.n_layers) return PYR_ERR_INVALID;
  if (layer != c->last_prefilled) return PYR_ERR_ORDER;
  *dev_scores = at<float>(c, c->lay.score);
  return PYR_OK;
}

pyr_status_t pyr_cache_lse(const pyr_cache_t* c, int32_t layer, const float** dev_lse) {
  if (!c || !dev_lse) return PYR_ERR_NULL;
  if (layer < 0 || layer >= c->cfg.n_layers) return PYR_ERR_INVALID;
  if (layer != c->last_prefilled) return PYR_ERR_ORDER;
  *dev_lse = at<float>(c, c->lay.lse);
  return PYR_OK;
}

pyr_status_t pyr_cache_kv(const pyr_cache_t* c, int32_t layer, void** dev_k, void** dev_v) {
  if (!c) return PYR_ERR_NULL;
  if (layer < 0 || layer >= c->cfg.n_layers) return PYR_ERR_INVALID;
  if (dev_k) *dev_k = c->base + c->lay.layers[layer].k_off;
  if (dev_v) *dev_v = c->base + c->lay.layers[layer].v_off;
  return PYR_OK;
}

pyr_status_t pyr_cache_status(pyr_cache_t* c, void* stream, int32_t* host_status) {
  if (!c || !host_status) return PYR_ERR_NULL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int word = 0;
  if (cudaMemcpyAsync(&word, at<int>(c, c->lay.status), sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess)
    return PYR_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return PYR_ERR_CUDA;
  *host_status = word;
  return word == 0 ? PYR_OK : PYR_ERR_TIMEOUT;
}

namespace {
// the selection of layer `layer` as both orderings launch it (the position buffers swap when the layer is done)
pyr::SelectArgs select_args(pyr_cache* c, int layer) {
  const LayerPlan& p = c->lay.layers[layer];
  int32_t* pos_in = at<int32_t>(c, c->pos_cur ? c->lay.pos1 : c->lay.pos0);
  int32_t* pos_out = at<int32_t>(c, c->pos_cur ? c->lay.pos0 : c->lay.pos1);
  pyr::SelectArgs sa;
  sa.score = at<float>(c, c->lay.score);
  sa.idx = at<int32_t>(c, c->lay.idx);
  sa.pos_in = layer == 0 ? nullptr : pos_in;
  sa.pos_out = pos_out;
  sa.B = c->cfg.batch; sa.G = c->cfg.sel_groups; sa.n = p.n_in; sa.c = p.c; sa.k = p.k;
  sa.reencode = (c->cfg.flags & PYR_FLAG_POS_REENCODE) ? 1 : 0;
  return sa;
}
}  // namespace

pyr_status_t pyr_prefill_layer(pyr_cache_t* c, int32_t layer, const void* q, const void* k, const void* v,
                               void* out, int64_t qsb, int64_t qsn, int64_t qsh, int64_t ksb, int64_t ksn,
                               int64_t ksh, int64_t osb, int64_t osn, int64_t osh, void* stream) {
  if (!c || !q || !k || !v || !out) return PYR_ERR_NULL;
  if (layer < 0 || layer >= c->cfg.n_layers) return PYR_ERR_INVALID;
  if (layer != c->next_layer || c->phase != 0) return PYR_ERR_ORDER;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int D = c->cfg.head_dim;
  if (qsh < D || ksh < D || osh < D || qsn < D || ksn < D || osn < D) return PYR_ERR_INVALID;
  if (c->cfg.dtype == PYR_BF16) {
    const uintptr_t m = reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(k) |
                        reinterpret_cast<uintptr_t>(v) | reinterpret_cast<uintptr_t>(out);
    if (m % 16 || (qsb | qsn | qsh | ksb | ksn | ksh | osb | osn | osh) % 8) return PYR_ERR_INVALID;
  }
  if (c->needs_init) {
    pyr_status_t st = device_init(c, s);
    if (st != PYR_OK) return st;
  }
  const LayerPlan& p = c->lay.layers[layer];
  pyr::PrefillArgs a;
  a.q = q; a.k = k; a.v = v; a.out = out;
  a.lse = at<float>(c, c->lay.lse);
  a.score = at<float>(c, c->lay.score);
  a.w = at<float>(c, c->lay.w) + (c->cfg.recent_len - (p.n_in - p.c));  // newest queries keep their weights
  a.qsb = qsb; a.qsn = qsn; a.qsh = qsh; a.ksb = ksb; a.ksn = ksn; a.ksh = ksh;
  a.osb = osb; a.osn = osn; a.osh = osh;
  a.B = c->cfg.batch; a.n = p.n_in; a.Hq = c->cfg.n_q_heads; a.Hkv = c->cfg.n_kv_heads; a.D = D;
  a.L = p.n_in - p.c; a.G = c->cfg.sel_groups;
  a.scale = c->scale; a.dtype = c->cfg.dtype;
  a.status = at<int>(c, c->lay.status);
  const bool want_tc = c->cfg.dtype == PYR_BF16 && !(c->cfg.flags & PYR_FLAG_CUDA_CORE_PREFILL);
  const bool tc_attn = want_tc && pyr::prefill_tc_supported(a);
  const bool tc_score = want_tc && pyr::score_tc_supported(a);
  cudaError_t e;
  c->sf_out = nullptr;
  if ((c->cfg.flags & PYR_FLAG_SELECT_FIRST) && tc_attn && tc_score && p.c > 0 && p.k < p.c) {
    // Select-first ordering: the query tiles that hold the window, the scores, the selection, and then the
    // rest of the tiles, whose rows go straight to their places among the kept rows.
    const int tiles = (p.n_in + 127) / 128, first_window_tile = p.c / 128;
    a.tile_k0 = 0; a.tile_k1 = tiles - first_window_tile;
    if (pyr::launch_prefill_tc(a, s) != cudaSuccess) return PYR_ERR_CUDA;
    if (pyr::launch_score_tc(a, at<float>(c, c->lay.score_part), s) != cudaSuccess) return PYR_ERR_CUDA;
    pyr::SelectArgs sa = select_args(c, layer);
    sa.rank = at<int32_t>(c, c->lay.rank);
    if (pyr::launch_select(sa, s) != cudaSuccess) return PYR_ERR_CUDA;
    a.tile_k0 = a.tile_k1; a.tile_k1 = 1 << 30; a.rank = sa.rank;
    if (pyr::launch_prefill_tc(a, s) != cudaSuccess) return PYR_ERR_CUDA;
    g_launches += first_window_tile > 0 ? 5 : 4;
    c->sf_out = out;
    c->sf_boundary = first_window_tile * 128;
  } else {
    e = tc_attn ? pyr::launch_prefill_tc(a, s) : pyr::launch_prefill_simt(a, s);
    if (e != cudaSuccess) return PYR_ERR_CUDA;
    g_launches += 1;
    if (p.c > 0) {
      e = tc_score ? pyr::launch_score_tc(a, at<float>(c, c->lay.score_part), s) : pyr::launch_score_simt(a, s);
      if (e != cudaSuccess) return PYR_ERR_CUDA;
      g_launches += tc_score ? 2 : 1;
    }
  }
  if (c->lay.q_ring > 0) {
    // the window's queries go to the layer's ring: the generation phase re-scores the cache with them
    const int eb = c->cfg.dtype == PYR_BF16 ? 2 : 4;
    const int Lw = p.n_in - p.c;
    const int64_t row_bytes = (int64_t)c->cfg.n_q_heads * D * eb;
    if (qsh != D || qsn != (int64_t)c->cfg.n_q_heads * D) return PYR_ERR_UNSUPPORTED;   // rows must be contiguous
    e = pyr::launch_copy_rows(static_cast<const char*>(q) + (int64_t)p.c * qsn * eb, c->base + p.q_off, qsb * eb,
                              qsn * eb, (int64_t)c->lay.q_ring * row_bytes, row_bytes, c->cfg.batch, Lw,
                              (int)row_bytes, s);
    if (e != cudaSuccess) return PYR_ERR_CUDA;
    g_launches += 1;
    c->q_count[layer] = Lw;
  }
  c->phase = 1;
  c->last_prefilled = layer;
  return PYR_OK;
}

pyr_status_t pyr_select_compact(pyr_cache_t* c, int32_t layer, const void* k, const void* v, int64_t ksb,
                                int64_t ksn, int64_t ksh, void* rows, int64_t row_elems, int64_t rsb,
                                int64_t rsn, int64_t rsg, int32_t* n_out, void* stream) {
  if (!c || !k || !v) return PYR_ERR_NULL;
  if (layer < 0 || layer >= c->cfg.n_layers) return PYR_ERR_INVALID;
  if (layer != c->next_layer || c->phase != 1) return PYR_ERR_ORDER;
  const int D = c->cfg.head_dim;
  const int eb = c->cfg.dtype == PYR_BF16 ? 2 : 4;
  if (ksh < D || ksn < D) return PYR_ERR_INVALID;
  if (reinterpret_cast<uintptr_t>(k) % 16 || reinterpret_cast<uintptr_t>(v) % 16 ||
      (ksb * eb) % 16 || (ksn * eb) % 16 || (ksh * eb) % 16)
    return PYR_ERR_INVALID;
  if (rows) {
    if (row_elems < 1 || rsn < row_elems) return PYR_ERR_INVALID;
    if (c->cfg.sel_groups == 1 ? rsg != 0 : rsg < 1) return PYR_ERR_INVALID;
    if (reinterpret_cast<uintptr_t>(rows) % 16 || (row_elems * eb) % 16 || (rsb * eb) % 16 ||
        (rsn * eb) % 16 || (rsg * eb) % 16)
      return PYR_ERR_INVALID;
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const LayerPlan& p = c->lay.layers[layer];
  const pyr::SelectArgs sa = select_args(c, layer);
  const bool selected = c->sf_out != nullptr;          // select-first ordering: the prefill call has run the selection
  if (!selected) {
    if (pyr::launch_select(sa, s) != cudaSuccess) return PYR_ERR_CUDA;
    g_launches += 1;
  }

  pyr::GatherArgs ga;
  ga.k = k; ga.v = v;
  ga.kc = c->base + p.k_off; ga.vc = c->base + p.v_off;
  ga.idx = sa.idx; ga.ksb = ksb; ga.ksn = ksn; ga.ksh = ksh;
  ga.B = c->cfg.batch; ga.Hkv = c->cfg.n_kv_heads; ga.G = c->cfg.sel_groups; ga.D = D;
  ga.n_out = p.n_out; ga.cap = p.cap; ga.elem_bytes = eb;
  if (pyr::launch_gather_kv(ga, s) != cudaSuccess) return PYR_ERR_CUDA;
  g_launches += 1;

  if (rows && p.n_out < p.n_in) {
    pyr::RowsArgs ra;
    ra.rows = rows; ra.idx = sa.idx; ra.stride_b = rsb; ra.stride_n = rsn; ra.stride_g = rsg;
    ra.row_elems = row_elems; ra.B = c->cfg.batch; ra.G = c->cfg.sel_groups; ra.n_out = p.n_out;
    ra.elem_bytes = eb;
    ra.idx_div = 1;
    if (selected && rows == c->sf_out) {
      // these are the rows the prefill call wrote: all but those of the tiles that held the window are in
      // place; a row moves up by at most the number of rows dropped
      ra.src_begin = c->sf_boundary;
      ra.dst_begin = c->sf_boundary - (p.n_in - p.n_out) > 0 ? c->sf_boundary - (p.n_in - p.n_out) : 0;
    }
    if (pyr::launch_compact_rows(ra, s) != cudaSuccess) return PYR_ERR_CUDA;
    g_launches += 1;
  }
  c->sf_out = nullptr;
  if (n_out) *n_out = p.n_out;
  c->len_now[layer] = p.n_out;
  c->pos_cur ^= 1;
  c->last_selected = layer;
  c->next_layer = layer + 1;
  c->phase = 0;
  return PYR_OK;
}

pyr_status_t pyr_decode_attn(pyr_cache_t* c, int32_t layer, const void* q, const void* k_new,
                             const void* v_new, void* out, void* stream) {
  if (!c || !q || !k_new || !v_new || !out) return PYR_ERR_NULL;
  if (layer < 0 || layer >= c->cfg.n_layers) return PYR_ERR_INVALID;
  if (c->next_layer != c->cfg.n_layers) return PYR_ERR_ORDER;
  const LayerPlan& p = c->lay.layers[layer];
  if (c->len_now[layer] >= p.cap) return PYR_ERR_CAPACITY;
  if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(k_new) |
       reinterpret_cast<uintptr_t>(v_new) | reinterpret_cast<uintptr_t>(out)) % 16)
    return PYR_ERR_INVALID;
  pyr::DecodeArgs a;
  a.q = q; a.k_new = k_new; a.v_new = v_new; a.out = out;
  a.kc = c->base + p.k_off; a.vc = c->base + p.v_off;
  a.part_acc = at<float>(c, c->lay.part_acc);
  a.part_ml = at<float>(c, c->lay.part_ml);
  a.B = c->cfg.batch; a.Hq = c->cfg.n_q_heads; a.Hkv = c->cfg.n_kv_heads; a.D = c->cfg.head_dim;
  a.len = c->len_now[layer]; a.cap = p.cap;
  a.scale = c->scale; a.dtype = c->cfg.dtype;
  a.status = at<int>(c, c->lay.status);
  a.spin_limit = c->wait_test_armed ? 4096u : 0u;
  a.skip_chunk = c->wait_test_armed ? 0 : -1;
  c->wait_test_armed = false;
  int splits = 1, rps = 0;
  const int sms = pyr::device_sm_count();
  if (sms <= 0) return PYR_ERR_CUDA;
  pyr::decode_split_rule(a.B, a.Hkv, a.len + 1, sms, &splits, &rps);
  a.splits = splits; a.rows_per_split = rps;
  if (pyr::launch_decode(a, static_cast<cudaStream_t>(stream)) != cudaSuccess) return PYR_ERR_CUDA;
  g_launches += splits > 1 ? 2 : 1;
  c->len_now[layer] += 1;
  if (c->lay.q_ring > 0) {
    const int eb = c->cfg.dtype == PYR_BF16 ? 2 : 4;
    const int64_t row_bytes = (int64_t)c->cfg.n_q_heads * c->cfg.head_dim * eb;
    const int slot = (int)(c->q_count[layer] % c->lay.q_ring);
    if (pyr::launch_copy_rows(q, c->base + p.q_off + (int64_t)slot * row_bytes, row_bytes, row_bytes,
                              (int64_t)c->lay.q_ring * row_bytes, row_bytes, c->cfg.batch, 1, (int)row_bytes,
                              static_cast<cudaStream_t>(stream)) != cudaSuccess)
      return PYR_ERR_CUDA;
    g_launches += 1;
    c->q_count[layer] += 1;
  }
  return PYR_OK;
}

// ---- decoder glue of whole-model workloads: argument checks and dispatch
static bool glue_ok(int32_t dtype, std::initializer_list<const void*> ptrs) {
  if (dtype != PYR_BF16 && dtype != PYR_F32) return false;
  for (const void* p : ptrs) if (!p) return false;
  return true;
}
#define PYR_GLUE(call) do { if ((call) != cudaSuccess) return PYR_ERR_CUDA; g_launches += 1; return PYR_OK; } while (0)

pyr_status_t pyr_glue_embed(const int32_t* ids, const void* table, void* out, int64_t tokens, int32_t d, int32_t vocab,
                            int32_t dtype, int32_t* dev_status, void* stream) {
  if (!glue_ok(dtype, {ids, table, out})) return dtype == PYR_BF16 || dtype == PYR_F32 ? PYR_ERR_NULL : PYR_ERR_UNSUPPORTED;
  if (tokens < 0 || d < 1 || vocab < 1) return PYR_ERR_INVALID;
  PYR_GLUE(pyr::launch_glue_embed(ids, table, out, tokens, d, vocab, dtype, dev_status, static_cast<cudaStream_t>(stream)));
}
namespace {
// a row list per sequence: every argument in range, the list's rows themselves are the caller's promise
bool row_map_ok(const int32_t* rows, int32_t batch, int32_t n_src, int32_t n_dst, int64_t rows_stride) {
  return rows && batch >= 0 && n_src >= 1 && n_dst >= 1 && rows_stride >= n_dst;
}
pyr::RowMap row_map(const int32_t* rows, int32_t n_src, int32_t n_dst, int64_t rows_stride) {
  pyr::RowMap m;
  m.rows = rows; m.rows_stride = rows_stride; m.n_src = n_src; m.n_dst = n_dst;
  return m;
}
}  // namespace

pyr_status_t pyr_glue_rmsnorm(const void* x, const void* gain, void* out, int64_t tokens, int32_t d, float eps,
                              int32_t dtype, void* stream) {
  if (!glue_ok(dtype, {x, gain, out})) return dtype == PYR_BF16 || dtype == PYR_F32 ? PYR_ERR_NULL : PYR_ERR_UNSUPPORTED;
  if (tokens < 0 || d < 1 || !(eps >= 0.f)) return PYR_ERR_INVALID;
  PYR_GLUE(pyr::launch_glue_rmsnorm(x, gain, out, tokens, d, eps, dtype, pyr::RowMap(), static_cast<cudaStream_t>(stream)));
}
pyr_status_t pyr_glue_rmsnorm_rows(const void* x, const int32_t* rows, int64_t rows_stride, const void* gain, void* out,
                                   int32_t batch, int32_t n_src, int32_t n_dst, int32_t d, float eps, int32_t dtype,
                                   void* stream) {
  if (!glue_ok(dtype, {x, rows, gain, out})) return dtype == PYR_BF16 || dtype == PYR_F32 ? PYR_ERR_NULL : PYR_ERR_UNSUPPORTED;
  if (!row_map_ok(rows, batch, n_src, n_dst, rows_stride) || d < 1 || !(eps >= 0.f)) return PYR_ERR_INVALID;
  PYR_GLUE(pyr::launch_glue_rmsnorm(x, gain, out, (int64_t)batch * n_dst, d, eps, dtype, row_map(rows, n_src, n_dst, rows_stride),
                                    static_cast<cudaStream_t>(stream)));
}
pyr_status_t pyr_glue_linear(const void* x, const void* w, const void* residual, void* y, int64_t m, int32_t n,
                             int32_t k, int32_t dtype, void* stream) {
  if (!glue_ok(dtype, {x, w, y})) return dtype == PYR_BF16 || dtype == PYR_F32 ? PYR_ERR_NULL : PYR_ERR_UNSUPPORTED;
  if (m < 0 || n < 1 || k < 1) return PYR_ERR_INVALID;
  if (m == 0) return PYR_OK;
  if (dtype == PYR_BF16 && pyr::gemm_skinny_supported(x, w, residual, y, m, n, k))
    PYR_GLUE(pyr::launch_gemm_skinny(x, w, residual, &y, 1, m, n, k, pyr::glue_status_word(), static_cast<cudaStream_t>(stream)));
  if (dtype == PYR_BF16 && pyr::gemm_tc_supported(x, w, residual, y, m, n, k))
    PYR_GLUE(pyr::launch_gemm_tc(x, w, residual, y, m, n, k, pyr::glue_status_word(), pyr::RowMap(), static_cast<cudaStream_t>(stream)));
  PYR_GLUE(pyr::launch_glue_linear(x, w, residual, y, m, n, k, dtype, pyr::RowMap(), static_cast<cudaStream_t>(stream)));
}
pyr_status_t pyr_glue_linear_split(const void* x, const void* w, void* const* ys, int32_t n_parts, int64_t m, int32_t part_n,
                                   int32_t k, int32_t dtype, void* stream) {
  if (!ys) return PYR_ERR_NULL;
  if (n_parts < 1 || n_parts > 4) return PYR_ERR_INVALID;
  for (int i = 0; i < n_parts; ++i)
    if (!ys[i]) return PYR_ERR_NULL;
  if (!glue_ok(dtype, {x, w})) return dtype == PYR_BF16 || dtype == PYR_F32 ? PYR_ERR_NULL : PYR_ERR_UNSUPPORTED;
  if (m < 0 || part_n < 1 || k < 1) return PYR_ERR_INVALID;
  if (m == 0) return PYR_OK;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int n = part_n * n_parts;
  bool aligned = true;
  for (int i = 0; i < n_parts; ++i) aligned = aligned && reinterpret_cast<uintptr_t>(ys[i]) % 16 == 0;
  if (dtype == PYR_BF16 && aligned && part_n % 128 == 0 && pyr::gemm_skinny_supported(x, w, nullptr, ys[0], m, n, k))
    PYR_GLUE(pyr::launch_gemm_skinny(x, w, nullptr, ys, n_parts, m, n, k, pyr::glue_status_word(), s));
  // otherwise one product per part, on the rows of w that belong to it
  const size_t eb = dtype == PYR_BF16 ? 2 : 4;
  for (int i = 0; i < n_parts; ++i) {
    const pyr_status_t st = pyr_glue_linear(x, static_cast<const char*>(w) + (size_t)i * part_n * k * eb, nullptr, ys[i], m, part_n, k,
                                            dtype, stream);
    if (st != PYR_OK) return st;
  }
  return PYR_OK;
}
pyr_status_t pyr_glue_linear_rows(const void* x, const void* w, const void* residual, const int32_t* res_rows,
                                  int64_t rows_stride, void* y, int32_t batch, int32_t n_src, int32_t n_dst, int32_t n,
                                  int32_t k, int32_t dtype, void* stream) {
  if (!glue_ok(dtype, {x, w, residual, res_rows, y})) return dtype == PYR_BF16 || dtype == PYR_F32 ? PYR_ERR_NULL : PYR_ERR_UNSUPPORTED;
  if (!row_map_ok(res_rows, batch, n_src, n_dst, rows_stride) || n < 1 || k < 1) return PYR_ERR_INVALID;
  const int64_t m = (int64_t)batch * n_dst;
  if (m == 0) return PYR_OK;
  const pyr::RowMap map = row_map(res_rows, n_src, n_dst, rows_stride);
  if (dtype == PYR_BF16 && pyr::gemm_tc_supported(x, w, residual, y, m, n, k))
    PYR_GLUE(pyr::launch_gemm_tc(x, w, residual, y, m, n, k, pyr::glue_status_word(), map, static_cast<cudaStream_t>(stream)));
  PYR_GLUE(pyr::launch_glue_linear(x, w, residual, y, m, n, k, dtype, map, static_cast<cudaStream_t>(stream)));
}
pyr_status_t pyr_glue_linear_swiglu(const void* x, const void* w_gate, const void* w_up, void* out, int64_t m, int32_t n,
                                    int32_t k, int32_t dtype, void* stream) {
  if (!glue_ok(dtype, {x, w_gate, w_up, out})) return dtype == PYR_BF16 || dtype == PYR_F32 ? PYR_ERR_NULL : PYR_ERR_UNSUPPORTED;
  if (m < 0 || n < 1 || k < 1) return PYR_ERR_INVALID;
  if (m == 0) return PYR_OK;
  if (dtype != PYR_BF16 || !pyr::gemm_tc_supported(x, w_gate, w_up, out, m, n, k)) return PYR_ERR_UNSUPPORTED;
  PYR_GLUE(pyr::launch_gemm_tc_gated(x, w_gate, w_up, out, m, n, k, pyr::glue_status_word(), static_cast<cudaStream_t>(stream)));
}
pyr_status_t pyr_glue_status(void* stream, int32_t* host_status) {
  if (!host_status) return PYR_ERR_NULL;
  int* word_dev = pyr::glue_status_word();
  if (!word_dev) return PYR_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int word = 0;
  const int zero = 0;
  if (cudaMemcpyAsync(&word, word_dev, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess) return PYR_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return PYR_ERR_CUDA;
  if (word != 0) {       // reported once, then the record starts clean
    if (cudaMemcpyAsync(word_dev, &zero, sizeof(int), cudaMemcpyHostToDevice, s) != cudaSuccess) return PYR_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return PYR_ERR_CUDA;
  }
  *host_status = word;
  return word == 0 ? PYR_OK : PYR_ERR_TIMEOUT;
}
pyr_status_t pyr_glue_rope(void* x, const int32_t* pos, int64_t tokens, int32_t n_heads, int32_t head_dim,
                           int32_t dtype, void* stream) {
  if (!glue_ok(dtype, {x, pos})) return dtype == PYR_BF16 || dtype == PYR_F32 ? PYR_ERR_NULL : PYR_ERR_UNSUPPORTED;
  if (tokens < 0 || n_heads < 1 || head_dim < 2 || head_dim % 2) return PYR_ERR_INVALID;
  if (head_dim > 256) return PYR_ERR_UNSUPPORTED;
  PYR_GLUE(pyr::launch_glue_rope(x, pos, tokens, n_heads, head_dim, dtype, static_cast<cudaStream_t>(stream)));
}
pyr_status_t pyr_glue_swiglu(const void* gate, const void* up, void* out, int64_t n, int32_t dtype, void* stream) {
  if (!glue_ok(dtype, {gate, up, out})) return dtype == PYR_BF16 || dtype == PYR_F32 ? PYR_ERR_NULL : PYR_ERR_UNSUPPORTED;
  if (n < 0) return PYR_ERR_INVALID;
  PYR_GLUE(pyr::launch_glue_swiglu(gate, up, out, n, dtype, static_cast<cudaStream_t>(stream)));
}
pyr_status_t pyr_glue_argmax(const void* x, int32_t* out, int64_t rows, int32_t n, int32_t dtype, void* stream) {
  if (!glue_ok(dtype, {x, out})) return dtype == PYR_BF16 || dtype == PYR_F32 ? PYR_ERR_NULL : PYR_ERR_UNSUPPORTED;
  if (rows < 0 || n < 1) return PYR_ERR_INVALID;
  PYR_GLUE(pyr::launch_glue_argmax(x, out, rows, n, dtype, static_cast<cudaStream_t>(stream)));
}

int32_t pyr_recent_len_from_ratio(int32_t prompt_len, double ratio) {
  if (prompt_len < 1 || !(ratio >= 0.0)) return 0;
  long long L = (long long)std::floor(ratio * (double)prompt_len);
  if (L < 1) L = 1;
  if (L > prompt_len) L = prompt_len;
  return (int32_t)L;
}

pyr_status_t pyr_cache_arm_wait_test(pyr_cache_t* c) {
  if (!c) return PYR_ERR_NULL;
  c->wait_test_armed = true;
  return PYR_OK;
}

pyr_status_t pyr_decode_reselect(pyr_cache_t* c, int32_t layer, int32_t* c_ctx, int32_t* n_out, void* stream) {
  if (!c) return PYR_ERR_NULL;
  if (layer < 0 || layer >= c->cfg.n_layers) return PYR_ERR_INVALID;
  if (c->lay.q_ring == 0) return PYR_ERR_UNSUPPORTED;
  if (c->next_layer != c->cfg.n_layers) return PYR_ERR_ORDER;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const LayerPlan& p = c->lay.layers[layer];
  const int L = c->cfg.recent_len;
  const int len = c->len_now[layer];
  const long long qn = c->q_count[layer];
  const int Lw = (int)(qn < L ? qn : L);
  const int ctx = len - Lw;
  if (c_ctx) *c_ctx = ctx;
  if (ctx <= p.k) {                       // Algorithm 1 selects only while the cache exceeds its bound
    if (n_out) *n_out = len;
    return PYR_OK;
  }
  const int eb = c->cfg.dtype == PYR_BF16 ? 2 : 4;
  const int D = c->cfg.head_dim;
  pyr::GenScoreArgs ga;
  ga.qwin = c->base + p.q_off; ga.kc = c->base + p.k_off;
  ga.part = at<float>(c, c->lay.gen_part); ga.score = at<float>(c, c->lay.score);
  ga.w = at<float>(c, c->lay.w) + (L - Lw);
  ga.B = c->cfg.batch; ga.Hq = c->cfg.n_q_heads; ga.Hkv = c->cfg.n_kv_heads; ga.D = D; ga.G = c->cfg.sel_groups;
  ga.R = c->lay.q_ring; ga.start = (int)((qn - Lw) % c->lay.q_ring); ga.Lw = Lw; ga.len = len; ga.cap = p.cap; ga.c = ctx;
  ga.scale = c->scale; ga.dtype = c->cfg.dtype;
  if (pyr::launch_gen_score(ga, s) != cudaSuccess) return PYR_ERR_CUDA;

  pyr::SelectArgs sa;
  sa.score = ga.score;
  sa.idx = at<int32_t>(c, c->lay.idx);
  sa.pos_in = nullptr;                    // positions are not tracked through the generation phase
  sa.pos_out = at<int32_t>(c, c->pos_cur ? c->lay.pos0 : c->lay.pos1);
  sa.B = c->cfg.batch; sa.G = c->cfg.sel_groups; sa.n = len; sa.c = ctx; sa.k = p.k;
  if (pyr::launch_select(sa, s) != cudaSuccess) return PYR_ERR_CUDA;
  c->pos_cur ^= 1;
  c->last_selected = layer;
  c->last_prefilled = layer;             // the score buffer now holds this layer's generation-phase scores

  // K and V rows move up in place: kept indices ascend, so a row's destination lies at or below its source
  pyr::RowsArgs ra;
  ra.idx = sa.idx; ra.stride_b = (int64_t)c->cfg.n_kv_heads * p.cap * D; ra.stride_n = D;
  ra.stride_g = (int64_t)p.cap * D; ra.row_elems = D; ra.B = c->cfg.batch; ra.G = c->cfg.n_kv_heads;
  ra.n_out = p.k + Lw; ra.elem_bytes = eb; ra.idx_div = c->cfg.n_kv_heads / c->cfg.sel_groups;
  ra.rows = c->base + p.k_off;
  if (pyr::launch_compact_rows(ra, s) != cudaSuccess) return PYR_ERR_CUDA;
  ra.rows = c->base + p.v_off;
  if (pyr::launch_compact_rows(ra, s) != cudaSuccess) return PYR_ERR_CUDA;
  g_launches += 5;
  c->len_now[layer] = p.k + Lw;
  if (n_out) *n_out = p.k + Lw;
  return PYR_OK;
}

}  // extern "C"
