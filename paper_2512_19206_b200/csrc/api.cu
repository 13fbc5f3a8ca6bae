// Host side of the C ABI: argument checking, the cache memory map, per-layer length tracking and the
// scheduling of the kernels.  No device allocation happens here.
#include <algorithm>
#include <new>
#include <vector>

#include "common.cuh"

using namespace mixkvq;

struct mixkvq_cache {
  mixkvq_config cfg;
  char* mem;
  size_t bytes;
  int S, g, R, G, U, NG, VG, max_blocks, tile;
  uint32_t base_bytes, unit_bytes;
  uint64_t extras_budget;
  // byte offsets inside one layer and per-stream strides
  uint64_t state_off, table_off, resk_off, resv_off, base_off, extras_off, sink_off, seq_off, layer_stride;
  uint64_t state_stride, table_stride, resk_stride, resv_stride, base_stride, extras_stride, sink_stride;
  // fill of every sequence of every layer, index layer * batch + b: packed blocks, tokens in the residual window, sink rows
  std::vector<int> n_blocks, r, n_sink;
  int n_sms;
  int attn_kind;
  uint64_t launches;
  // What the library enqueued last on this handle: kNoPackedWrite if it did not write packed blocks, a layer index if
  // it wrote that layer's packed blocks (a flush), kAllPacked after initialisation, a reset or a write from outside.
  // The next decode attention on such a layer waits for all earlier work before it reads anything.
  int last_packed_writer;
  uint32_t test_extra_tx, test_wait_polls;   // mixkvq_test_arm_copy_timeout
};

namespace {

constexpr uint64_t kHeaderBytes = 256;   // device status word lives at offset 0
constexpr int kNoPackedWrite = -1, kAllPacked = -2;

uint64_t align_up(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }

int check_config(const mixkvq_config* c) {
  if (!c) return MIXKVQ_E_INVALID_ARG;
  if (c->n_layers < 1 || c->batch < 1 || c->n_q_heads < 1 || c->n_kv_heads < 1 || c->max_tokens < 1)
    return MIXKVQ_E_INVALID_ARG;
  if (c->n_q_heads % c->n_kv_heads != 0) return MIXKVQ_E_INVALID_ARG;
  if (c->head_dim != kD || (c->v_bits != 2 && c->v_bits != 4)) return MIXKVQ_E_UNSUPPORTED;
  if (c->v_bits == 4 && c->block_layout != 0) return MIXKVQ_E_UNSUPPORTED;      // the tile layout holds 2-bit values only
  if (c->n_q_heads / c->n_kv_heads > 8) return MIXKVQ_E_UNSUPPORTED;
  if (c->group_size != 32 && c->group_size != 64 && c->group_size != 128) return MIXKVQ_E_UNSUPPORTED;
  if (c->residual_len < 32 || c->residual_len > 256 || c->residual_len % 32 != 0 ||
      c->residual_len % c->group_size != 0)
    return MIXKVQ_E_UNSUPPORTED;
  if (c->score_bits != 2 && c->score_bits != 4) return MIXKVQ_E_UNSUPPORTED;
  if (c->importance_mode < 0 || c->importance_mode > 2) return MIXKVQ_E_INVALID_ARG;
  if (c->block_layout != 0 && c->block_layout != 1) return MIXKVQ_E_INVALID_ARG;
  if (c->budget_bf16 < 0 || c->budget_u4 < 0 || c->budget_bf16 + c->budget_u4 > kD) return MIXKVQ_E_INVALID_ARG;
  if (c->sink_len < 0 || c->sink_len > 256 || c->sink_len % 32 != 0 || c->reserved != 0) return MIXKVQ_E_INVALID_ARG;
  if (c->block_layout == 1 && c->residual_len != 128) return MIXKVQ_E_UNSUPPORTED;
  return MIXKVQ_OK;
}

// Fills the geometry and the memory map; returns total bytes.
uint64_t plan(const mixkvq_config* c, mixkvq_cache* h) {
  h->cfg = *c;
  h->S = c->batch * c->n_kv_heads;
  h->g = c->n_q_heads / c->n_kv_heads;
  h->R = c->residual_len;
  h->G = c->group_size;
  h->U = h->R / 32;
  h->NG = h->R / h->G;
  h->VG = kD / h->G;
  h->max_blocks = (c->max_tokens + h->R - 1) / h->R;
  h->unit_bytes = 2048u + 128u * h->VG + (c->v_bits == 4 ? 1024u : 0u);
  h->tile = (c->block_layout == 1) ? 1 : 0;
  h->base_bytes = h->tile ? (uint32_t)h->NG * 512u + 8192u + 512u * (uint32_t)h->VG
                          : (uint32_t)h->NG * 512u + (uint32_t)h->U * h->unit_bytes;
  h->extras_budget = c->extras_budget_bytes ? align_up(c->extras_budget_bytes, 16)
                                            : align_up((uint64_t)h->max_blocks * h->R * 32, 256);
  h->state_stride = kStateBytes;
  h->table_stride = align_up((uint64_t)h->max_blocks * 8, 256);
  h->resk_stride = (uint64_t)h->R * 256;
  h->resv_stride = (uint64_t)h->R * 256;
  h->base_stride = (uint64_t)h->max_blocks * h->base_bytes;
  h->extras_stride = align_up(h->extras_budget, 256);
  h->sink_stride = (uint64_t)c->sink_len * 512;      // keys then values, 256 bytes a row
  uint64_t off = 0;
  h->state_off = off;  off = align_up(off + h->state_stride * h->S, 256);
  h->table_off = off;  off = align_up(off + h->table_stride * h->S, 256);
  h->resk_off = off;   off = align_up(off + h->resk_stride * h->S, 256);
  h->resv_off = off;   off = align_up(off + h->resv_stride * h->S, 256);
  h->base_off = off;   off = align_up(off + h->base_stride * h->S, 256);
  h->extras_off = off; off = align_up(off + h->extras_stride * h->S, 256);
  h->sink_off = off;   off = align_up(off + h->sink_stride * h->S, 256);
  h->seq_off = off;    off = align_up(off + (uint64_t)c->batch * 16 + (uint64_t)(c->batch + 1) * 4, 256);
  h->layer_stride = off;
  return kHeaderBytes + h->layer_stride * (uint64_t)c->n_layers;
}

size_t workspace_bytes(int S) { return (size_t)(kMaxCtas + 2 * S) * kPartialFloats * sizeof(float); }

inline int fi(const mixkvq_cache* h, int layer, int b) { return layer * h->cfg.batch + b; }

bool same_fill(const mixkvq_cache* h, int layer, int b1, int b2) {
  const int i = fi(h, layer, b1), j = fi(h, layer, b2);
  return h->n_blocks[i] == h->n_blocks[j] && h->r[i] == h->r[j] && h->n_sink[i] == h->n_sink[j];
}
// every sequence of the layer holds the same number of blocks, residual tokens and sink rows
bool uniform(const mixkvq_cache* h, int layer) {
  for (int b = 1; b < h->cfg.batch; ++b)
    if (!same_fill(h, layer, 0, b)) return false;
  return true;
}
bool all_empty(const mixkvq_cache* h, int layer) {
  for (int b = 0; b < h->cfg.batch; ++b) {
    const int i = fi(h, layer, b);
    if (h->n_blocks[i] || h->r[i] || h->n_sink[i]) return false;
  }
  return true;
}
long long tokens_held(const mixkvq_cache* h, int layer, int b) {
  const int i = fi(h, layer, b);
  return (long long)h->n_sink[i] + (long long)h->n_blocks[i] * h->R + h->r[i];
}
long long max_tokens_held(const mixkvq_cache* h, int layer) {
  long long m = 0;
  for (int b = 0; b < h->cfg.batch; ++b) m = std::max(m, tokens_held(h, layer, b));
  return m;
}

// The layer's arrays for sequences b0 .. b0 + nb - 1 (all of them when nb < 0), which share the fill of sequence b0.
LayerView view(const mixkvq_cache* h, int layer, int b0 = 0, int nb = -1) {
  LayerView v{};
  v.B = nb < 0 ? h->cfg.batch : nb; v.Hq = h->cfg.n_q_heads; v.Hkv = h->cfg.n_kv_heads; v.g = h->g;
  v.R = h->R; v.G = h->G; v.U = h->U; v.NG = h->NG; v.VG = h->VG;
  v.max_blocks = h->max_blocks;
  v.n_blocks = h->n_blocks[fi(h, layer, b0)]; v.r = h->r[fi(h, layer, b0)];
  v.tile = h->tile;
  v.budget_bf16 = h->cfg.budget_bf16; v.budget_u4 = h->cfg.budget_u4;
  v.v_bits = h->cfg.v_bits;
  v.dense_hi = (h->cfg.tau_u4 < 0.0f && v.budget_bf16 + v.budget_u4 == 0) ? 1 : 0;
  v.base_bytes = h->base_bytes; v.unit_bytes = h->unit_bytes;
  v.extras_budget = h->extras_budget;
  v.score_bits = h->cfg.score_bits; v.importance_mode = h->cfg.importance_mode;
  v.tau_bf16 = h->cfg.tau_bf16; v.tau_u4 = h->cfg.tau_u4;
  char* L = h->mem + kHeaderBytes + h->layer_stride * (uint64_t)layer;
  const uint64_t s0 = (uint64_t)b0 * h->cfg.n_kv_heads;      // first stream of the view
  v.state = L + h->state_off + s0 * h->state_stride;    v.state_stride = h->state_stride;
  v.table = L + h->table_off + s0 * h->table_stride;    v.table_stride = h->table_stride;
  v.resk = L + h->resk_off + s0 * h->resk_stride;       v.resk_stride = h->resk_stride;
  v.resv = L + h->resv_off + s0 * h->resv_stride;       v.resv_stride = h->resv_stride;
  v.base = L + h->base_off + s0 * h->base_stride;       v.base_stride = h->base_stride;
  v.extras = L + h->extras_off + s0 * h->extras_stride; v.extras_stride = h->extras_stride;
  v.sink = L + h->sink_off + s0 * h->sink_stride;       v.sink_stride = h->sink_stride;
  v.sink_len = h->cfg.sink_len; v.n_sink = h->n_sink[fi(h, layer, b0)];
  v.status = reinterpret_cast<uint32_t*>(h->mem);
  v.debug_extra_tx = h->test_extra_tx;
  v.wait_polls = h->test_wait_polls;
  return v;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int zero_layer_state(mixkvq_cache* h, int layer, cudaStream_t st) {
  char* L = h->mem + kHeaderBytes + h->layer_stride * (uint64_t)layer;
  if (cudaMemsetAsync(L + h->state_off, 0, h->state_stride * h->S, st) != cudaSuccess) return MIXKVQ_E_CUDA;
  for (int b = 0; b < h->cfg.batch; ++b) h->n_blocks[fi(h, layer, b)] = h->r[fi(h, layer, b)] = h->n_sink[fi(h, layer, b)] = 0;
  h->last_packed_writer = kAllPacked;
  return MIXKVQ_OK;
}

// Ragged batch: writes the fills of the layer's sequences to its table in device memory (as kernel arguments: ordered
// in the stream, no copy) and points the view at it.
int upload_seq_table(mixkvq_cache* h, int layer, cudaStream_t st, LayerView* lv) {
  const int B = h->cfg.batch;
  if (B > kMaxRaggedBatch) return MIXKVQ_E_UNSUPPORTED;
  SeqTableArgs a{};
  a.n = B;
  a.Hkv = h->cfg.n_kv_heads;
  long long total = 0;
  for (int b = 0; b < B; ++b) {
    const int i = fi(h, layer, b);
    a.fill[3 * b] = h->n_blocks[i];
    a.fill[3 * b + 1] = h->r[i];
    a.fill[3 * b + 2] = h->n_sink[i];
    a.w[b] = attention_ws_positions_of(h->n_blocks[i], h->r[i], h->n_sink[i], h->U);
    total += (long long)a.Hkv * a.w[b];
  }
  if (total >= (1ll << 31)) return MIXKVQ_E_UNSUPPORTED;
  char* L = h->mem + kHeaderBytes + h->layer_stride * (uint64_t)layer + h->seq_off;
  int4* seq = reinterpret_cast<int4*>(L);
  int* prefix = reinterpret_cast<int*>(L + (size_t)B * 16);
  if (launch_seq_table(a, seq, prefix, st) != cudaSuccess) return MIXKVQ_E_CUDA;
  h->launches += 1;
  lv->seq = seq;
  lv->seq_prefix = prefix;
  lv->seq_total = total;
  return MIXKVQ_OK;
}

// Picks the decode-attention kernel for the layer's layout and the selected kind, enqueues it and counts its launches.
int run_attention(mixkvq_cache* h, int layer, const void* q, float* out, float scale, float* ws, cudaStream_t st,
                  const void* new_k = nullptr, const void* new_v = nullptr, float* lse = nullptr) {
  LayerView lv = view(h, layer);
  lv.new_k = static_cast<const uint16_t*>(new_k);
  lv.new_v = static_cast<const uint16_t*>(new_v);
  lv.stage_early = (h->last_packed_writer == kNoPackedWrite ||
                    (h->last_packed_writer >= 0 && h->last_packed_writer != layer)) ? 1 : 0;
  h->last_packed_writer = kNoPackedWrite;
  if (!uniform(h, layer)) {
    // ragged batch: the split kernel and the merge walk every stream's own positions
    if (h->tile || h->attn_kind == 1) return MIXKVQ_E_UNSUPPORTED;
    const int rc = upload_seq_table(h, layer, st, &lv);
    if (rc != MIXKVQ_OK) return rc;
    lv.stage_early = 0;
  }
  int launches = 0;
  cudaError_t e;
  if (h->attn_kind == 1)
    e = launch_attention_simt(lv, q, out, scale, ws, h->n_sms, st, &launches);
  else if (h->tile)
    e = launch_attention_tc(lv, q, h->attn_kind == 2 ? nullptr : out, scale, ws, h->n_sms, st, &launches);
  else
    e = launch_attention_ws(lv, q, h->attn_kind == 2 ? nullptr : out, scale, ws, h->n_sms, st, &launches, lse);
  h->launches += launches;
  return e == cudaSuccess ? MIXKVQ_OK : MIXKVQ_E_CUDA;
}

// Appends tokens 0 .. n_tokens - 1 of the tensors (whose token dimension is n_stride long) to sequences b0 .. b0 + nb - 1,
// which share one fill: sink rows first, then flush / bulk blocks / residual rows as the fill demands.
int append_run_first(mixkvq_cache* cache, int layer, int b0, int nb, const void* k_dev, const void* v_dev, const void* q_dev,
                     int n_stride, int n_tokens, cudaStream_t st) {
  const char* k = static_cast<const char*>(k_dev) + (size_t)b0 * cache->cfg.n_kv_heads * n_stride * kD * 2;
  const char* v = static_cast<const char*>(v_dev) + (size_t)b0 * cache->cfg.n_kv_heads * n_stride * kD * 2;
  const char* q = static_cast<const char*>(q_dev) + (size_t)b0 * cache->cfg.n_q_heads * n_stride * kD * 2;
  // the run's fill is kept in the first sequence's slots here; append_run copies it to the others
  int& sink0 = cache->n_sink[fi(cache, layer, b0)];
  int& r0 = cache->r[fi(cache, layer, b0)];
  int& nb0 = cache->n_blocks[fi(cache, layer, b0)];
  int t = 0;
  while (t < n_tokens) {
    if (sink0 < cache->cfg.sink_len) {
      // the first tokens of the sequence are sink tokens: stored as they are, outside everything else
      const int room = cache->cfg.sink_len - sink0;
      const int m = n_tokens - t < room ? n_tokens - t : room;
      LayerView lv = view(cache, layer, b0, nb);
      if (launch_sink_append(lv, k, v, n_stride, t, m, st) != cudaSuccess) return MIXKVQ_E_CUDA;
      cache->launches += 1;
      cache->last_packed_writer = kNoPackedWrite;
      sink0 += m;
      t += m;
      continue;
    }
    if (r0 == cache->R) {
      LayerView lv = view(cache, layer, b0, nb);
      if (launch_flush(lv, st) != cudaSuccess) return MIXKVQ_E_CUDA;
      cache->launches += 1;
      cache->last_packed_writer = layer;
      nb0 += 1;
      r0 = 0;
    }
    // prefill: complete windows go straight from the tensors to packed blocks; the last 1..R tokens stay in the
    // residual window
    if (r0 == 0 && n_tokens - t > cache->R) {
      int nblk = (n_tokens - t - 1) / cache->R;
      if (nblk > 32768) nblk = 32768;                  // grid.y limit
      LayerView lv = view(cache, layer, b0, nb);
      if (launch_flush_bulk(lv, k, v, q, n_stride, t, nblk, st) != cudaSuccess) return MIXKVQ_E_CUDA;
      cache->launches += cache->cfg.importance_mode == 1 ? 4 : 3;
      cache->last_packed_writer = layer;
      nb0 += nblk;
      t += nblk * cache->R;
      continue;
    }
    const int m = (n_tokens - t < cache->R - r0) ? n_tokens - t : cache->R - r0;
    LayerView lv = view(cache, layer, b0, nb);
    if (launch_append(lv, k, v, q, n_stride, t, m, st) != cudaSuccess) return MIXKVQ_E_CUDA;
    cache->launches += 1;
    cache->last_packed_writer = kNoPackedWrite;
    r0 += m;
    t += m;
  }
  return MIXKVQ_OK;
}

int append_run(mixkvq_cache* cache, int layer, int b0, int nb, const void* k_dev, const void* v_dev, const void* q_dev,
               int n_stride, int n_tokens, cudaStream_t st) {
  const int rc = append_run_first(cache, layer, b0, nb, k_dev, v_dev, q_dev, n_stride, n_tokens, st);
  for (int b = b0 + 1; b < b0 + nb; ++b) {
    cache->n_sink[fi(cache, layer, b)] = cache->n_sink[fi(cache, layer, b0)];
    cache->r[fi(cache, layer, b)] = cache->r[fi(cache, layer, b0)];
    cache->n_blocks[fi(cache, layer, b)] = cache->n_blocks[fi(cache, layer, b0)];
  }
  return rc;
}

}  // namespace

extern "C" {

int mixkvq_cache_bytes(const mixkvq_config* cfg, size_t* cache_bytes, size_t* attn_workspace_bytes) {
  int rc = check_config(cfg);
  if (rc != MIXKVQ_OK) return rc;
  mixkvq_cache tmp{};
  uint64_t total = plan(cfg, &tmp);
  if (cache_bytes) *cache_bytes = (size_t)total;
  if (attn_workspace_bytes) *attn_workspace_bytes = workspace_bytes(tmp.S);
  return MIXKVQ_OK;
}

int mixkvq_cache_init(const mixkvq_config* cfg, void* cache_dev, size_t bytes, void* stream, mixkvq_cache** out) {
  int rc = check_config(cfg);
  if (rc != MIXKVQ_OK) return rc;
  if (!cache_dev || !out) return MIXKVQ_E_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(cache_dev) & 255u) return MIXKVQ_E_ALIGNMENT;
  mixkvq_cache* h = new (std::nothrow) mixkvq_cache();
  if (!h) return MIXKVQ_E_INVALID_ARG;
  uint64_t total = plan(cfg, h);
  if (bytes < total) { delete h; return MIXKVQ_E_BUFFER_TOO_SMALL; }
  h->mem = static_cast<char*>(cache_dev);
  h->bytes = bytes;
  h->n_blocks.assign((size_t)cfg->n_layers * cfg->batch, 0);
  h->r.assign((size_t)cfg->n_layers * cfg->batch, 0);
  h->n_sink.assign((size_t)cfg->n_layers * cfg->batch, 0);
  h->attn_kind = 0;
  h->launches = 0;
  h->last_packed_writer = kAllPacked;
  h->test_extra_tx = h->test_wait_polls = 0;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&h->n_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
    delete h;
    return MIXKVQ_E_CUDA;
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(h->mem, 0, kHeaderBytes, st) != cudaSuccess) { delete h; return MIXKVQ_E_CUDA; }
  for (int l = 0; l < cfg->n_layers; ++l)
    if (zero_layer_state(h, l, st) != MIXKVQ_OK) { delete h; return MIXKVQ_E_CUDA; }
  if (attention_ws_setup() != cudaSuccess || attention_tc_setup() != cudaSuccess || prefill_attention_setup() != cudaSuccess) { delete h; return MIXKVQ_E_CUDA; }
  *out = h;
  return MIXKVQ_OK;
}

int mixkvq_cache_destroy(mixkvq_cache* cache) {
  delete cache;
  return MIXKVQ_OK;
}

int mixkvq_cache_reset(mixkvq_cache* cache, int layer, void* stream) {
  if (!cache || layer >= cache->cfg.n_layers) return MIXKVQ_E_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (layer >= 0) return zero_layer_state(cache, layer, st);
  cache->last_packed_writer = kAllPacked;
  if (cudaMemsetAsync(cache->mem, 0, kHeaderBytes, st) != cudaSuccess) return MIXKVQ_E_CUDA;
  for (int l = 0; l < cache->cfg.n_layers; ++l)
    if (zero_layer_state(cache, l, st) != MIXKVQ_OK) return MIXKVQ_E_CUDA;
  return MIXKVQ_OK;
}

int mixkvq_select_channels(mixkvq_cache* cache, int layer, uint8_t* tiers_dev, double* salience_dev, void* stream) {
  if (!cache || !tiers_dev || layer < 0 || layer >= cache->cfg.n_layers) return MIXKVQ_E_INVALID_ARG;
  bool any = false;
  for (int b = 0; b < cache->cfg.batch; ++b) any = any || cache->r[fi(cache, layer, b)] > 0;
  if (!any) return MIXKVQ_E_EMPTY;
  cache->last_packed_writer = kNoPackedWrite;
  // one launch per run of sequences with the same fill (one launch for a batch of equal lengths); a sequence whose
  // window is empty has no scores: its rows of the outputs are left as they are
  const int B = cache->cfg.batch, Hkv = cache->cfg.n_kv_heads;
  for (int b0 = 0; b0 < B;) {
    int b1 = b0 + 1;
    while (b1 < B && same_fill(cache, layer, b0, b1)) ++b1;
    if (cache->r[fi(cache, layer, b0)] > 0) {
      LayerView lv = view(cache, layer, b0, b1 - b0);
      if (launch_select_window(lv, tiers_dev + (size_t)b0 * Hkv * kD, salience_dev ? salience_dev + (size_t)b0 * Hkv * kD : nullptr,
                               static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return MIXKVQ_E_CUDA;
      cache->launches += 1;
    }
    b0 = b1;
  }
  return MIXKVQ_OK;
}

int mixkvq_select_channels_raw(const void* q_dev, const void* k_dev, int batch, int n_q_heads, int n_kv_heads,
                               int lq, int lk, int score_bits, float tau_bf16, float tau_u4,
                               uint8_t* tiers_dev, double* salience_dev, void* stream) {
  if (!q_dev || !k_dev || !tiers_dev || batch < 1 || n_q_heads < 1 || n_kv_heads < 1 || lq < 1 || lk < 1 ||
      n_q_heads % n_kv_heads != 0)
    return MIXKVQ_E_INVALID_ARG;
  if (score_bits != 2 && score_bits != 4) return MIXKVQ_E_UNSUPPORTED;
  return launch_select_raw(q_dev, k_dev, batch, n_q_heads, n_kv_heads, lq, lk, score_bits, tau_bf16, tau_u4,
                           tiers_dev, salience_dev, static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? MIXKVQ_OK : MIXKVQ_E_CUDA;
}

int mixkvq_quantize_append(mixkvq_cache* cache, int layer, const void* k_dev, const void* v_dev, const void* q_dev,
                           int n_tokens, void* stream) {
  if (!cache || n_tokens < 1) return MIXKVQ_E_INVALID_ARG;
  std::vector<int32_t> counts((size_t)cache->cfg.batch, n_tokens);
  return mixkvq_quantize_append_ragged(cache, layer, k_dev, v_dev, q_dev, n_tokens, counts.data(), stream);
}

int mixkvq_quantize_append_ragged(mixkvq_cache* cache, int layer, const void* k_dev, const void* v_dev, const void* q_dev,
                                  int n_tokens_max, const int32_t* n_tokens_host, void* stream) {
  if (!cache || !k_dev || !v_dev || !q_dev || !n_tokens_host || layer < 0 || layer >= cache->cfg.n_layers || n_tokens_max < 1)
    return MIXKVQ_E_INVALID_ARG;
  if (!aligned16(k_dev) || !aligned16(v_dev) || !aligned16(q_dev)) return MIXKVQ_E_ALIGNMENT;
  const int B = cache->cfg.batch;
  for (int b = 0; b < B; ++b) {
    if (n_tokens_host[b] < 0 || n_tokens_host[b] > n_tokens_max) return MIXKVQ_E_INVALID_ARG;
    if (tokens_held(cache, layer, b) + n_tokens_host[b] > cache->cfg.max_tokens) return MIXKVQ_E_CAPACITY;
  }
  // runs of neighbouring sequences with the same fill and the same number of new tokens go through the kernels together
  // (a batch of equal lengths is one run)
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  for (int b0 = 0; b0 < B;) {
    int b1 = b0 + 1;
    while (b1 < B && n_tokens_host[b1] == n_tokens_host[b0] && same_fill(cache, layer, b0, b1)) ++b1;
    if (n_tokens_host[b0] > 0) {
      const int rc = append_run(cache, layer, b0, b1 - b0, k_dev, v_dev, q_dev, n_tokens_max, n_tokens_host[b0], st);
      if (rc != MIXKVQ_OK) return rc;
    }
    b0 = b1;
  }
  return MIXKVQ_OK;
}

int mixkvq_decode_attention(mixkvq_cache* cache, int layer, const void* q_dev, float* out_dev, float softmax_scale,
                            void* workspace_dev, size_t workspace_bytes_given, void* stream) {
  if (!cache || !q_dev || !out_dev || !workspace_dev || layer < 0 || layer >= cache->cfg.n_layers)
    return MIXKVQ_E_INVALID_ARG;
  if (!aligned16(q_dev) || !aligned16(out_dev) || !aligned16(workspace_dev)) return MIXKVQ_E_ALIGNMENT;
  if (workspace_bytes_given < workspace_bytes(cache->S)) return MIXKVQ_E_BUFFER_TOO_SMALL;
  if (all_empty(cache, layer)) return MIXKVQ_E_EMPTY;
  return run_attention(cache, layer, q_dev, out_dev, softmax_scale, static_cast<float*>(workspace_dev),
                       static_cast<cudaStream_t>(stream));
}

int mixkvq_decode_attention_partial(mixkvq_cache* cache, int layer, const void* q_dev, float* out_dev, float* lse_dev,
                                    float softmax_scale, void* workspace_dev, size_t workspace_bytes_given, void* stream) {
  if (!cache || !q_dev || !out_dev || !lse_dev || !workspace_dev || layer < 0 || layer >= cache->cfg.n_layers)
    return MIXKVQ_E_INVALID_ARG;
  if (!aligned16(q_dev) || !aligned16(out_dev) || !aligned16(workspace_dev)) return MIXKVQ_E_ALIGNMENT;
  if (workspace_bytes_given < workspace_bytes(cache->S)) return MIXKVQ_E_BUFFER_TOO_SMALL;
  if (cache->tile || cache->attn_kind != 0) return MIXKVQ_E_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (all_empty(cache, layer)) {
    // this cache holds no token of the context: weight 0 in the merge
    cache->launches += 1;
    return launch_empty_partial(out_dev, lse_dev, cache->cfg.batch * cache->cfg.n_q_heads, st) == cudaSuccess
               ? MIXKVQ_OK : MIXKVQ_E_CUDA;
  }
  return run_attention(cache, layer, q_dev, out_dev, softmax_scale, static_cast<float*>(workspace_dev), st, nullptr, nullptr,
                       lse_dev);
}

int mixkvq_merge_partials(const float* o_parts_dev, const float* lse_parts_dev, int n_parts, int rows, float* out_dev,
                          void* stream) {
  if (!o_parts_dev || !lse_parts_dev || !out_dev || n_parts < 1 || n_parts > 1024 || rows < 1) return MIXKVQ_E_INVALID_ARG;
  if (!aligned16(o_parts_dev) || !aligned16(out_dev)) return MIXKVQ_E_ALIGNMENT;
  return launch_merge_partials(o_parts_dev, lse_parts_dev, n_parts, rows, out_dev, static_cast<cudaStream_t>(stream)) ==
                 cudaSuccess ? MIXKVQ_OK : MIXKVQ_E_CUDA;
}

int mixkvq_decode_step(mixkvq_cache* cache, int layer, const void* k_dev, const void* v_dev, const void* q_dev,
                       float* out_dev, float softmax_scale, void* workspace_dev, size_t workspace_bytes_given,
                       void* stream) {
  if (!cache || !k_dev || !v_dev || !q_dev || !out_dev || !workspace_dev || layer < 0 || layer >= cache->cfg.n_layers)
    return MIXKVQ_E_INVALID_ARG;
  if (!aligned16(k_dev) || !aligned16(v_dev) || !aligned16(q_dev) || !aligned16(out_dev) || !aligned16(workspace_dev))
    return MIXKVQ_E_ALIGNMENT;
  if (workspace_bytes_given < workspace_bytes(cache->S)) return MIXKVQ_E_BUFFER_TOO_SMALL;
  if (max_tokens_held(cache, layer) + 1 > cache->cfg.max_tokens) return MIXKVQ_E_CAPACITY;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int B = cache->cfg.batch;
  bool sink_room = false;
  for (int b = 0; b < B; ++b) sink_room = sink_room || cache->n_sink[fi(cache, layer, b)] < cache->cfg.sink_len;
  if (cache->attn_kind != 0 || sink_room) {
    // the comparison kernels do not take the new token themselves, and a sink token is not a residual token:
    // plain append, then attention
    int rc = mixkvq_quantize_append(cache, layer, k_dev, v_dev, q_dev, 1, stream);
    if (rc != MIXKVQ_OK) return rc;
    return run_attention(cache, layer, q_dev, out_dev, softmax_scale, static_cast<float*>(workspace_dev), st);
  }
  // full windows are flushed first: one launch; in a ragged batch the kernel reads the fills from the layer's table and
  // only the sequences whose window is full take part
  bool any_full = false;
  for (int b = 0; b < B; ++b) any_full = any_full || cache->r[fi(cache, layer, b)] == cache->R;
  if (any_full) {
    LayerView lv = view(cache, layer);
    if (!uniform(cache, layer)) {
      if (cache->tile) return MIXKVQ_E_UNSUPPORTED;
      const int rc = upload_seq_table(cache, layer, st, &lv);
      if (rc != MIXKVQ_OK) return rc;
    }
    if (launch_flush(lv, st) != cudaSuccess) return MIXKVQ_E_CUDA;
    cache->launches += 1;
    cache->last_packed_writer = layer;
    for (int b = 0; b < B; ++b)
      if (cache->r[fi(cache, layer, b)] == cache->R) {
        cache->n_blocks[fi(cache, layer, b)] += 1;
        cache->r[fi(cache, layer, b)] = 0;
      }
  }
  for (int b = 0; b < B; ++b) cache->r[fi(cache, layer, b)] += 1;   // the attention kernel stores the token at slot r - 1 and accumulates |q|
  const int rc = run_attention(cache, layer, q_dev, out_dev, softmax_scale, static_cast<float*>(workspace_dev), st, k_dev, v_dev);
  if (rc != MIXKVQ_OK)
    for (int b = 0; b < B; ++b) cache->r[fi(cache, layer, b)] -= 1;   // nothing was enqueued: the token is not part of the layer
  return rc;
}

size_t mixkvq_prefill_scratch_bytes(const mixkvq_config* cfg, int n_tokens) {
  if (check_config(cfg) != MIXKVQ_OK || n_tokens < 1) return 0;
  return prefill_scratch_bytes(cfg->batch, cfg->n_kv_heads, n_tokens);
}

int mixkvq_prefill(mixkvq_cache* cache, int layer, const void* k_dev, const void* v_dev, const void* q_dev, int n_tokens,
                   float* out_dev, float softmax_scale, void* scratch_dev, size_t scratch_bytes, void* stream) {
  if (!cache || !k_dev || !v_dev || !q_dev || !out_dev || !scratch_dev || layer < 0 || layer >= cache->cfg.n_layers ||
      n_tokens < 1 || !(softmax_scale > 0.f))
    return MIXKVQ_E_INVALID_ARG;
  if (!aligned16(k_dev) || !aligned16(v_dev) || !aligned16(q_dev) || !aligned16(out_dev) || !aligned16(scratch_dev))
    return MIXKVQ_E_ALIGNMENT;
  // the prompt attends to itself only: the layer must be empty
  if (!all_empty(cache, layer)) return MIXKVQ_E_UNSUPPORTED;
  if (n_tokens > cache->cfg.max_tokens ||
      scratch_bytes < prefill_scratch_bytes(cache->cfg.batch, cache->cfg.n_kv_heads, n_tokens))
    return MIXKVQ_E_CAPACITY;
  if (launch_prefill_attention(q_dev, k_dev, v_dev, out_dev, scratch_dev, cache->cfg.batch, cache->cfg.n_q_heads,
                               cache->cfg.n_kv_heads, n_tokens, softmax_scale, reinterpret_cast<uint32_t*>(cache->mem),
                               cache->test_wait_polls, cache->test_extra_tx, static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return MIXKVQ_E_CUDA;
  cache->launches += 2;
  cache->last_packed_writer = kNoPackedWrite;
  return mixkvq_quantize_append(cache, layer, k_dev, v_dev, q_dev, n_tokens, stream);
}

int mixkvq_rope_append(mixkvq_cache* cache, int layer, void* k_dev, const void* v_dev, void* q_dev, const float* cos_dev,
                       const float* sin_dev, int pos0, int n_tokens, void* stream) {
  if (!cache || !k_dev || !v_dev || !q_dev || !cos_dev || !sin_dev || layer < 0 || layer >= cache->cfg.n_layers ||
      n_tokens < 1 || pos0 < 0)
    return MIXKVQ_E_INVALID_ARG;
  if (!aligned16(k_dev) || !aligned16(v_dev) || !aligned16(q_dev) || !aligned16(cos_dev) || !aligned16(sin_dev))
    return MIXKVQ_E_ALIGNMENT;
  if (max_tokens_held(cache, layer) + n_tokens > cache->cfg.max_tokens) return MIXKVQ_E_CAPACITY;      // nothing is rotated either
  if (launch_rope(k_dev, q_dev, cos_dev, sin_dev, cache->cfg.batch, cache->cfg.n_kv_heads, cache->cfg.n_q_heads, n_tokens,
                  pos0, static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return MIXKVQ_E_CUDA;
  cache->launches += 1;
  cache->last_packed_writer = kNoPackedWrite;
  return mixkvq_quantize_append(cache, layer, k_dev, v_dev, q_dev, n_tokens, stream);
}

int mixkvq_rope_decode_step(mixkvq_cache* cache, int layer, void* k_dev, const void* v_dev, void* q_dev,
                            const float* cos_dev, const float* sin_dev, int pos, float* out_dev, float softmax_scale,
                            void* workspace_dev, size_t workspace_bytes_given, void* stream) {
  if (!cache || !k_dev || !v_dev || !q_dev || !cos_dev || !sin_dev || !out_dev || !workspace_dev || layer < 0 ||
      layer >= cache->cfg.n_layers || pos < 0)
    return MIXKVQ_E_INVALID_ARG;
  if (!aligned16(k_dev) || !aligned16(v_dev) || !aligned16(q_dev) || !aligned16(cos_dev) || !aligned16(sin_dev) ||
      !aligned16(out_dev) || !aligned16(workspace_dev))
    return MIXKVQ_E_ALIGNMENT;
  if (workspace_bytes_given < workspace_bytes(cache->S)) return MIXKVQ_E_BUFFER_TOO_SMALL;
  if (max_tokens_held(cache, layer) + 1 > cache->cfg.max_tokens) return MIXKVQ_E_CAPACITY;
  if (launch_rope(k_dev, q_dev, cos_dev, sin_dev, cache->cfg.batch, cache->cfg.n_kv_heads, cache->cfg.n_q_heads, 1, pos,
                  static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return MIXKVQ_E_CUDA;
  cache->launches += 1;
  cache->last_packed_writer = kNoPackedWrite;
  return mixkvq_decode_step(cache, layer, k_dev, v_dev, q_dev, out_dev, softmax_scale, workspace_dev, workspace_bytes_given,
                            stream);
}

// ---- decode attention with the split partials in storage compiled into the library (no allocation)
namespace {
constexpr size_t kBuiltinScratchBytes =
    (size_t)(kMaxCtas + 2 * MIXKVQ_NOALLOC_MAX_STREAMS) * kPartialFloats * sizeof(float);
constexpr int kMaxDevices = 64;
}  // namespace
// In host code this name is only a handle for cudaGetSymbolAddress, never a device pointer.
static __device__ __align__(256) unsigned char g_builtin_scratch[kBuiltinScratchBytes];
static void* g_builtin_scratch_addr[kMaxDevices];      // device address of the array, per device ordinal

int mixkvq_decode_attention_noalloc(mixkvq_cache* cache, int layer, const void* q_dev, float* out_dev,
                                    float softmax_scale, void* stream) {
  if (!cache || !q_dev || !out_dev || layer < 0 || layer >= cache->cfg.n_layers) return MIXKVQ_E_INVALID_ARG;
  if (!aligned16(q_dev) || !aligned16(out_dev)) return MIXKVQ_E_ALIGNMENT;
  if (cache->S > MIXKVQ_NOALLOC_MAX_STREAMS) return MIXKVQ_E_BUILTIN_SCRATCH;
  if (all_empty(cache, layer)) return MIXKVQ_E_EMPTY;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MIXKVQ_E_CUDA;
  // the scratch array of the CURRENT device is used: it must be the device that holds the cache memory
  cudaPointerAttributes attr;
  if (cudaPointerGetAttributes(&attr, cache->mem) != cudaSuccess) return MIXKVQ_E_CUDA;
  if (attr.type != cudaMemoryTypeDevice || attr.device != dev) return MIXKVQ_E_INVALID_ARG;
  if (!g_builtin_scratch_addr[dev]) {
    // once per device, with that device current: resolve the array's address on this device
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_builtin_scratch) != cudaSuccess || !p) return MIXKVQ_E_CUDA;
    g_builtin_scratch_addr[dev] = p;
  }
  return run_attention(cache, layer, q_dev, out_dev, softmax_scale, static_cast<float*>(g_builtin_scratch_addr[dev]),
                       static_cast<cudaStream_t>(stream));
}

int mixkvq_cache_written_externally(mixkvq_cache* cache) {
  if (!cache) return MIXKVQ_E_INVALID_ARG;
  cache->last_packed_writer = kAllPacked;
  return MIXKVQ_OK;
}

int mixkvq_test_arm_copy_timeout(mixkvq_cache* cache, uint32_t extra_bytes, uint32_t max_polls) {
  if (!cache || (extra_bytes & 15u)) return MIXKVQ_E_INVALID_ARG;
  cache->test_extra_tx = extra_bytes;
  cache->test_wait_polls = max_polls;
  return MIXKVQ_OK;
}

int mixkvq_set_attention_kernel(mixkvq_cache* cache, int kind) {
  if (!cache || kind < 0 || kind > 2) return MIXKVQ_E_INVALID_ARG;
  cache->attn_kind = kind;
  return MIXKVQ_OK;
}

int mixkvq_query_status(mixkvq_cache* cache, int* device_status, void* stream) {
  if (!cache || !device_status) return MIXKVQ_E_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint32_t w = 0;
  if (cudaMemcpyAsync(&w, cache->mem, sizeof(w), cudaMemcpyDeviceToHost, st) != cudaSuccess) return MIXKVQ_E_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return MIXKVQ_E_CUDA;
  *device_status = (int)w;
  return MIXKVQ_OK;
}

int mixkvq_cache_describe(const mixkvq_cache* cache, int layer, mixkvq_layout_desc* out) {
  if (!cache || !out || layer < 0 || layer >= cache->cfg.n_layers) return MIXKVQ_E_INVALID_ARG;
  const uint64_t L = kHeaderBytes + cache->layer_stride * (uint64_t)layer;
  out->state_off = L + cache->state_off;   out->state_stride = cache->state_stride;
  out->table_off = L + cache->table_off;   out->table_stride = cache->table_stride;
  out->resk_off = L + cache->resk_off;     out->resk_stride = cache->resk_stride;
  out->resv_off = L + cache->resv_off;     out->resv_stride = cache->resv_stride;
  out->base_off = L + cache->base_off;     out->base_stride = cache->base_stride;
  out->extras_off = L + cache->extras_off; out->extras_stride = cache->extras_stride;
  out->base_bytes = cache->base_bytes;
  out->max_blocks = (uint32_t)cache->max_blocks;
  out->n_streams = (uint32_t)cache->S;
  out->n_blocks = (uint32_t)cache->n_blocks[fi(cache, layer, 0)];
  out->residual_tokens = (uint32_t)cache->r[fi(cache, layer, 0)];
  out->sink_off = L + cache->sink_off;     out->sink_stride = cache->sink_stride;
  out->sink_tokens = (uint32_t)cache->n_sink[fi(cache, layer, 0)];
  out->sink_len = (uint32_t)cache->cfg.sink_len;
  return MIXKVQ_OK;
}

int mixkvq_sequence_fill(const mixkvq_cache* cache, int layer, int b, uint32_t* n_blocks, uint32_t* residual_tokens,
                         uint32_t* sink_tokens) {
  if (!cache || layer < 0 || layer >= cache->cfg.n_layers || b < 0 || b >= cache->cfg.batch) return MIXKVQ_E_INVALID_ARG;
  if (n_blocks) *n_blocks = (uint32_t)cache->n_blocks[fi(cache, layer, b)];
  if (residual_tokens) *residual_tokens = (uint32_t)cache->r[fi(cache, layer, b)];
  if (sink_tokens) *sink_tokens = (uint32_t)cache->n_sink[fi(cache, layer, b)];
  return MIXKVQ_OK;
}

uint64_t mixkvq_launch_count(const mixkvq_cache* cache) { return cache ? cache->launches : 0; }

const char* mixkvq_status_string(int status) {
  switch (status) {
    case MIXKVQ_OK: return "ok";
    case MIXKVQ_E_INVALID_ARG: return "invalid argument";
    case MIXKVQ_E_UNSUPPORTED: return "unsupported configuration";
    case MIXKVQ_E_ALIGNMENT: return "device pointer not 16-byte aligned";
    case MIXKVQ_E_BUFFER_TOO_SMALL: return "cache memory or workspace too small";
    case MIXKVQ_E_CAPACITY: return "append exceeds max_tokens";
    case MIXKVQ_E_CUDA: return "CUDA error";
    case MIXKVQ_E_EMPTY: return "layer holds no tokens";
    case MIXKVQ_E_BUILTIN_SCRATCH: return "batch * n_kv_heads exceeds the built-in scratch (MIXKVQ_NOALLOC_MAX_STREAMS)";
    default: return "unknown status";
  }
}

}  // extern "C"
