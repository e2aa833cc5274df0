// Host runtime behind the C ABI: paged store (free list + chunk table), per-call integer plan
// (hit test, page allocation, slot/position/row arrays, gather items, attention tiles), kernel
// launches on the caller's stream, commit of missed chunks after success.
#include <algorithm>
#include <chrono>
#include <functional>
#include <cstring>
#include <new>
#include <unordered_map>
#include <vector>

#include "../../include/percache.h"
#include "kernels.h"

using namespace pc;

namespace {

struct ChunkEntry {
  int32_t n_tokens;
  std::vector<int32_t> pages;
  int64_t retrievals = 1;     // prompts that used this chunk (the one that stored it included)
  uint64_t serial = 0;        // insertion order
};

struct LayerWeights {
  __half *wqkv = nullptr, *wo = nullptr, *wgu = nullptr, *wd = nullptr;
  float *g_attn = nullptr, *g_ffn = nullptr;
  GemmOperand m_wqkv, m_wo, m_wgu, m_wd;                  // B maps with 128-row boxes
  GemmOperand m_wqkv256, m_wo256, m_wgu256, m_wd256;      // and with 256-row boxes
  AttnMaps attn_maps;
  AttnMaps paged_maps;                                    // paper-faithful mode: Q, K, V pages of this layer
  AttnMaps gf_maps;                                       // gather-free default mode: query buffer + V pages
};

struct Plan {   // integer description of the last successful call (host)
  std::vector<int32_t> cu_ctx, cu_new, slot_chunk, slot_offset, slot_is_new, row_slot;
  std::vector<int32_t> ctx0;      // device context slot of every prompt's slot 0 (prompts are decode_reserve apart)
  std::vector<int32_t> dec_len;   // tokens appended to every prompt by percache_decode since the prefill
  bool ctx_assembled = true;      // false after a gather-free call: there is no contiguous context to read or extend
  // gather-free call with a decode reserve: the prompts' page tables (8-entry padded) and where each starts, kept so
  // that the first decode step can assemble the context after all
  std::vector<int32_t> page_table, pt0;
};

constexpr int MAX_EVENTS = 1024;
constexpr int64_t GATHER_OVERLAP_MIN_BYTES = 512ll << 20;   // below this the per-layer waits cost more than they hide
constexpr int64_t GATHER_FREE_MIN_RATIO = 8;                // cached tokens per new row from which the fetch is skipped...
constexpr int64_t GATHER_FREE_MAX_NEW_ROWS = 256;           // ...if no prompt has more new rows than two attention tiles

// Key of a path of chunk ids (prefix mode): fold the ids with a 64-bit mixer (the SplitMix64 output function).
constexpr uint64_t PATH_KEY_SEED = 0x70657263616368ull;
inline uint64_t path_key_step(uint64_t path, uint64_t id) {
  uint64_t z = (path ^ id) + 0x9E3779B97F4A7C15ull + (path << 6) + (path >> 2);
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

}  // namespace

struct percache {
  percache_config_t cfg{};
  ModelDims dims{};
  cudaStream_t stream = nullptr;
  int n_sms = 148;
  uint32_t flags = 0;
  int gu_blk = 64;                          // gate/up interleave block (half the GEMM's N tile)

  std::vector<void*> dev_allocs;
  std::vector<LayerWeights> layers;
  float2* rope = nullptr;
  __nv_bfloat16 *kpool = nullptr, *vpool = nullptr;    // [L][pool_pages][16][kv_dim]
  __nv_bfloat16* qpool = nullptr;                       // paper-faithful mode only: [L][pool_pages][16][q_dim]
  bool paper_mode = false;
  __half *kctx = nullptr, *vctx = nullptr;              // [L][ctx_cap][kv_dim]
  float* resid = nullptr;                               // [m_cap][d]
  __nv_bfloat16* xin = nullptr;                         // [m_cap][d]
  __half *xn = nullptr, *qbuf = nullptr, *attn_out = nullptr, *act = nullptr;
  float* cref = nullptr;                                // reference kernels only
  float *partial_o = nullptr, *partial_ml = nullptr;    // attention parts of split tiles
  int partial_slots = 0;
  size_t max_attn_items = 0, max_attn_merges = 0;
  GemmOperand m_xn, m_attn, m_act;
  int64_t m_cap = 0, ctx_cap = 0;

  // index block: host (pinned) mirror and device copy
  int32_t* h_index = nullptr;
  int32_t* d_index = nullptr;
  size_t index_ints = 0;
  int* d_err = nullptr;
  int* h_err = nullptr;

  std::unordered_map<uint64_t, ChunkEntry> table;
  std::vector<int32_t> free_pages;
  int64_t store_limit = 0;     // pages the store may use (<= pool_pages)
  uint64_t next_serial = 0;

  Plan plan;
  std::vector<int32_t> retained_scratch;   // pages of rows that are not stored, kept for that late assembly
  float* capture_host = nullptr;   // debugging aid: layer inputs of the next calls are copied here (see header)
  int64_t capture_capacity = 0;    // floats
  int32_t decode_reserve = 0;     // context slots kept free behind every prompt for percache_decode
  percache_stats_t stats{};
  std::vector<cudaEvent_t> events;
  cudaEvent_t ev_begin = nullptr, ev_end = nullptr;
  // gather / compute overlap: the per-layer gathers of a large fetch run on `side`, layer l's
  // attention waits for ev_gather[l]
  cudaStream_t side = nullptr;
  cudaEvent_t ev_fork = nullptr;
  std::vector<cudaEvent_t> ev_gather;
};

namespace {

template <typename T>
bool dev_alloc(percache* h, T** out, size_t count) {
  void* p = nullptr;
  if (cudaMalloc(&p, std::max<size_t>(count * sizeof(T), 256)) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  h->dev_allocs.push_back(p);
  *out = static_cast<T*>(p);
  return true;
}

void destroy_impl(percache* h) {
  if (!h) return;
  cudaSetDevice(h->cfg.device);
  cudaStreamSynchronize(h->stream);
  for (void* p : h->dev_allocs) cudaFree(p);
  if (h->h_index) cudaFreeHost(h->h_index);
  if (h->h_err) cudaFreeHost(h->h_err);
  for (cudaEvent_t e : h->events)
    if (e) cudaEventDestroy(e);
  if (h->ev_begin) cudaEventDestroy(h->ev_begin);
  if (h->ev_end) cudaEventDestroy(h->ev_end);
  if (h->side) {
    cudaStreamSynchronize(h->side);
    cudaStreamDestroy(h->side);
  }
  if (h->ev_fork) cudaEventDestroy(h->ev_fork);
  for (cudaEvent_t e : h->ev_gather)
    if (e) cudaEventDestroy(e);
  cudaGetLastError();
  delete h;
}

// a bf16 matrix that may live on the host: copy to `tmp` on the device if so; returns what to read
const __nv_bfloat16* stage_bf16(const void* src, size_t elems, int on_device, __nv_bfloat16* tmp, cudaStream_t s,
                                bool* ok) {
  if (on_device) return static_cast<const __nv_bfloat16*>(src);
  if (cudaMemcpyAsync(tmp, src, elems * 2, cudaMemcpyHostToDevice, s) != cudaSuccess) *ok = false;
  return tmp;
}

struct PhaseTimer {
  percache* h;
  bool on;
  size_t next = 0;
  std::vector<int> phase_of;
  explicit PhaseTimer(percache* hh) : h(hh), on((hh->flags & PERCACHE_FLAG_PHASE_TIMING) != 0) {}
  bool room() const { return on && next + 2 <= h->events.size(); }
  void begin(int phase) {
    h->stats.phase_launches[phase]++;
    if (!room()) return;
    cudaEventRecord(h->events[next], h->stream);
    phase_of.push_back(phase);
  }
  void end() {
    if (!room()) return;
    cudaEventRecord(h->events[next + 1], h->stream);
    next += 2;
  }
  void collect() {
    for (size_t i = 0; i < next; i += 2) {
      float ms = 0.f;
      if (cudaEventElapsedTime(&ms, h->events[i], h->events[i + 1]) == cudaSuccess)
        h->stats.phase_us[phase_of[i / 2]] += 1000.0 * ms;
    }
  }
};

int alloc_pages(percache* h, int n, std::vector<int32_t>* out) {
  if (static_cast<size_t>(n) > h->free_pages.size()) return PERCACHE_E_NOSPACE;
  for (int i = 0; i < n; ++i) {
    out->push_back(h->free_pages.back());
    h->free_pages.pop_back();
  }
  return PERCACHE_OK;
}
void release_pages(percache* h, const std::vector<int32_t>& pages) {
  for (auto p = pages.rbegin(); p != pages.rend(); ++p) h->free_pages.push_back(*p);
}
void refresh_page_stats(percache* h) {
  h->stats.pages_free = static_cast<int64_t>(h->free_pages.size());
  h->stats.pages_used = h->cfg.pool_pages - h->stats.pages_free;
}

// Pages in use by stored chunks.
int64_t pages_in_use(const percache* h) { return h->cfg.pool_pages - static_cast<int64_t>(h->free_pages.size()); }

// Which chunks would have to go so that `need` more pages fit under the limit.  Nothing changes here.  Without the
// LFU flag this only checks.  With it, victims are taken least-frequently-used first (ties: oldest first), never a
// chunk whose id is in `keep`, and none unless the whole request can be met.  Returns the number of victims, or a
// negative code.
int pick_victims(const percache* h, int64_t need, const std::unordered_map<uint64_t, int64_t>& keep,
                 std::vector<uint64_t>* victims) {
  victims->clear();
  int64_t over = pages_in_use(h) + need - h->store_limit;
  if (over <= 0) return 0;
  if (!(h->flags & PERCACHE_FLAG_EVICT_LFU)) return PERCACHE_E_NOSPACE;
  std::vector<std::pair<std::pair<int64_t, uint64_t>, uint64_t>> order;     // ((count, serial), id)
  for (const auto& kv : h->table)
    if (!keep.count(kv.first)) order.push_back({{kv.second.retrievals, kv.second.serial}, kv.first});
  std::sort(order.begin(), order.end());
  size_t n_evict = 0;
  for (; n_evict < order.size() && over > 0; ++n_evict)
    over -= static_cast<int64_t>(h->table.find(order[n_evict].second)->second.pages.size());
  if (over > 0) return PERCACHE_E_NOSPACE;
  for (size_t i = 0; i < n_evict; ++i) victims->push_back(order[i].second);
  return static_cast<int>(n_evict);
}

// Pages of a call that stores chunks, taken so that the call can still be undone.  New pages come from the free
// list first and then from the pages of the chosen victims, which stay in the table until apply(): a call that
// fails on the host before that gives its free-list pages back (undo_host) and the store is exactly as it was.
// apply() is called right before the first kernel that writes pages; from then on the victims are gone and a
// failure only returns the new pages (undo_device).
struct PageTxn {
  percache* h;
  std::vector<uint64_t> victims;
  std::vector<int32_t> victim_pages, from_free, from_victims;
  bool applied = false;
  explicit PageTxn(percache* hh) : h(hh) {}
  void set_victims(const std::vector<uint64_t>& v) {
    victims = v;
    for (uint64_t id : v) {
      const ChunkEntry& e = h->table.find(id)->second;
      victim_pages.insert(victim_pages.end(), e.pages.begin(), e.pages.end());
    }
  }
  int take(int n, std::vector<int32_t>* out) {
    for (int i = 0; i < n; ++i) {
      if (!h->free_pages.empty()) {
        from_free.push_back(h->free_pages.back());
        out->push_back(h->free_pages.back());
        h->free_pages.pop_back();
      } else if (from_victims.size() < victim_pages.size()) {
        const int32_t pg = victim_pages[from_victims.size()];
        from_victims.push_back(pg);
        out->push_back(pg);
      } else {
        return PERCACHE_E_NOSPACE;
      }
    }
    return PERCACHE_OK;
  }
  void undo_host() {          // before apply(): the free list gets its pages back in the order they left
    for (auto p = from_free.rbegin(); p != from_free.rend(); ++p) h->free_pages.push_back(*p);
    from_free.clear();
    from_victims.clear();
  }
  void apply() {
    for (uint64_t id : victims) h->table.erase(id);
    for (size_t i = from_victims.size(); i < victim_pages.size(); ++i) h->free_pages.push_back(victim_pages[i]);
    applied = true;
  }
  void undo_device() {        // after apply(): the new pages return to the free list, the victims stay evicted
    for (auto p = from_victims.rbegin(); p != from_victims.rend(); ++p) h->free_pages.push_back(*p);
    for (auto p = from_free.rbegin(); p != from_free.rend(); ++p) h->free_pages.push_back(*p);
    from_free.clear();
    from_victims.clear();
  }
  void undo() { if (applied) undo_device(); else undo_host(); }
};

// upload a page list through the pinned index block and run `fn` with the device pointer
template <typename Fn>
int with_chunk_pages(percache* h, const std::vector<int32_t>& pages, Fn fn) {
  if (pages.size() > h->index_ints) return PERCACHE_E_CAPACITY;
  std::memcpy(h->h_index, pages.data(), pages.size() * sizeof(int32_t));
  if (cudaMemcpyAsync(h->d_index, h->h_index, pages.size() * sizeof(int32_t), cudaMemcpyHostToDevice, h->stream) !=
      cudaSuccess)
    return PERCACHE_E_CUDA;
  fn(h->d_index);
  if (cudaStreamSynchronize(h->stream) != cudaSuccess || cudaGetLastError() != cudaSuccess) return PERCACHE_E_CUDA;
  return PERCACHE_OK;
}

// Device-side index arrays of a call (inside h->d_index, same layout as the host block).
struct DevIndex {
  const int32_t *row_slot, *row_pos, *row_pool, *row_ctx0;
  const GatherItem* items;
  const AttnItem* attn_items;
  const int32_t* cta_first;
  const AttnMerge* merges;
};
DevIndex dev_index(const percache* h) {
  DevIndex ix;
  ix.row_slot = h->d_index;
  ix.row_pos = ix.row_slot + h->m_cap;
  ix.row_pool = ix.row_pos + h->m_cap;
  ix.row_ctx0 = ix.row_pool + h->m_cap;
  ix.items = reinterpret_cast<const GatherItem*>(ix.row_ctx0 + h->m_cap);
  ix.attn_items = reinterpret_cast<const AttnItem*>(reinterpret_cast<const int32_t*>(ix.items) + 4 * h->ctx_cap);
  ix.cta_first = reinterpret_cast<const int32_t*>(ix.attn_items) + 8 * h->max_attn_items;
  ix.merges = reinterpret_cast<const AttnMerge*>(ix.cta_first + h->n_sms + 1);
  return ix;
}

// Every decoder block for the Mi rows in h->resid (prefill: the new rows of the batch; decode: one row per
// prompt): RMSNorm, QKV projection (rotation, pages, context), attention over the assembled context, output
// projection, RMSNorm, SwiGLU FFN.  Layer l's attention first waits for ev_gather[l] when the fetch runs beside.
// n_decode_items > 0: the attention work is a decode step's list of DecodeAttnItem / DecodeAttnMerge records.
bool run_layers(percache* h, int Mi, const DevIndex& ix, int n_attn_ctas, int n_merges, bool overlap_gather,
                bool use_ref, PhaseTimer& timer, cudaStream_t s, int n_decode_items = 0,
                const int32_t* gather_free_page_table = nullptr) {
  const ModelDims& D = h->dims;
  const int d = D.d_model;
  const size_t pool_layer = static_cast<size_t>(h->cfg.pool_pages) * PAGE_TOKENS * D.kv_dim;
  const size_t ctx_layer = static_cast<size_t>(h->ctx_cap) * D.kv_dim;
  // CTA pairs: chosen per GEMM by size (see umma_gemm_pick_shape)
  const bool may_pair = !(h->flags & PERCACHE_FLAG_SINGLE_CTA_GEMM);
  const int32_t *d_row_slot = ix.row_slot, *d_row_pos = ix.row_pos, *d_row_pool = ix.row_pool, *d_row_ctx0 = ix.row_ctx0;
  const AttnItem* d_attn_items = ix.attn_items;
  const int32_t* d_cta_first = ix.cta_first;
  const AttnMerge* d_merges = ix.merges;
  // A handful of rows (decode) is a matter of reading the weights once: CUDA-core kernels bound by HBM, with the
  // RMSNorm folded into the QKV and gate/up projections
  const bool small_rows = !use_ref && !(h->flags & PERCACHE_FLAG_NO_SMALL_ROW_KERNELS) && Mi <= SMALL_GEMM_MAX_ROWS &&
                          (gather_free_page_table == nullptr || n_decode_items > 0) &&
                          d % 256 == 0 && D.q_dim % 256 == 0 && D.d_ffn % 256 == 0;
  bool ok = true;
  // debugging aid: the residual stream as it enters layer l goes to capture_host[l] (stream order does the rest)
  auto capture = [&](int l) {
    if (h->capture_host && static_cast<int64_t>(l + 1) * Mi * d <= h->capture_capacity)
      ok = ok && cudaMemcpyAsync(h->capture_host + static_cast<size_t>(l) * Mi * d, h->resid,
                                 static_cast<size_t>(Mi) * d * sizeof(float), cudaMemcpyDeviceToHost, s) == cudaSuccess;
  };
  for (int l = 0; l < D.n_layers && ok && Mi > 0; ++l) {
    LayerWeights& W = h->layers[l];
    capture(l);
    if (!small_rows) {
      timer.begin(PERCACHE_PH_NORM);
      launch_rmsnorm(h->resid, W.g_attn, h->xn, Mi, d, D.rms_eps, s);
      timer.end();
    }

    QkvEpilogue qe{};
    qe.rows = RowIndex{d_row_slot, d_row_pos, d_row_pool};
    qe.rope = h->rope;
    qe.q_out = h->qbuf;
    qe.kpool = h->kpool + l * pool_layer;
    qe.vpool = h->vpool + l * pool_layer;
    qe.kctx = h->kctx + l * ctx_layer;
    qe.vctx = h->vctx + l * ctx_layer;
    qe.n_q_heads = D.n_q_heads;
    qe.n_kv_heads = D.n_kv_heads;
    qe.skip_ctx = gather_free_page_table != nullptr ? 1 : 0;
    timer.begin(PERCACHE_PH_QKV);
    if (small_rows) {
      ok = ok && launch_small_gemm(EPI_QKV, &qe, Mi, D.qkv_dim, d, h->resid, W.g_attn, D.rms_eps, nullptr, W.wqkv, 0,
                                   h->n_sms, s) == 0;
    } else if (use_ref) {
      launch_ref_gemm(h->xn, W.wqkv, h->cref, Mi, D.qkv_dim, d, s);
      launch_ref_qkv_epilogue(h->cref, Mi, qe, s);
    } else {
      {
        int bn, ks, pr;
        umma_gemm_pick_shape(Mi, D.qkv_dim, d, h->n_sms, false, may_pair, &bn, &ks, &pr);
        ok = ok && launch_umma_gemm(h->m_xn, (bn == 256 && !pr) ? W.m_wqkv256 : W.m_wqkv, Mi, D.qkv_dim, d, bn, EPI_QKV, &qe, nullptr,
                                    h->d_err, h->n_sms, s, ks, pr) == 0;
      }
    }
    timer.end();

    timer.begin(PERCACHE_PH_ATTN);
    if (overlap_gather) ok = ok && cudaStreamWaitEvent(s, h->ev_gather[l], 0) == cudaSuccess;
    if (use_ref || (h->flags & PERCACHE_FLAG_REFERENCE_ATTENTION)) {
      launch_ref_attention(h->qbuf, qe.kctx, qe.vctx, h->attn_out, d_row_pos, d_row_ctx0, Mi, D.n_q_heads, D.n_kv_heads, s);
    } else if (n_decode_items > 0) {
      ok = ok && launch_decode_attention(reinterpret_cast<const DecodeAttnItem*>(d_attn_items), n_decode_items,
                                         reinterpret_cast<const DecodeAttnMerge*>(d_merges), n_merges, h->qbuf, qe.kctx,
                                         qe.vctx, h->partial_o, h->partial_ml, h->attn_out, D.n_q_heads, D.n_kv_heads,
                                         s, gather_free_page_table ? qe.kpool : nullptr,
                                         gather_free_page_table ? qe.vpool : nullptr, gather_free_page_table,
                                         h->rope) == 0;
    } else if (gather_free_page_table != nullptr) {
      // K and V straight from the pages (K rotated on load): no assembled context
      ok = ok && launch_umma_attention(W.gf_maps, d_attn_items, d_cta_first, n_attn_ctas, d_row_pos, h->attn_out,
                                       h->partial_o, h->partial_ml, D.n_q_heads, D.n_kv_heads, h->d_err, s,
                                       gather_free_page_table, 2, h->rope, h->cfg.max_prompt_tokens) == 0;
      launch_attention_merge(d_merges, n_merges, h->partial_o, h->partial_ml, h->attn_out, D.n_q_heads, D.n_kv_heads, s);
    } else {
      ok = ok && launch_umma_attention(W.attn_maps, d_attn_items, d_cta_first, n_attn_ctas, d_row_pos, h->attn_out,
                                       h->partial_o, h->partial_ml, D.n_q_heads, D.n_kv_heads, h->d_err, s) == 0;
      launch_attention_merge(d_merges, n_merges, h->partial_o, h->partial_ml, h->attn_out, D.n_q_heads, D.n_kv_heads, s);
    }
    timer.end();

    ResidualEpilogue re{h->resid, d};
    timer.begin(PERCACHE_PH_OPROJ);
    if (small_rows) {
      ok = ok && launch_small_gemm(EPI_RESIDUAL, &re, Mi, d, D.q_dim, nullptr, nullptr, 0.f, h->attn_out, W.wo, 0,
                                   h->n_sms, s) == 0;
    } else if (use_ref) {
      launch_ref_gemm(h->attn_out, W.wo, h->cref, Mi, d, D.q_dim, s);
      launch_ref_residual_epilogue(h->cref, Mi, d, re, s);
    } else {
      {
        int bn, ks, pr;
        umma_gemm_pick_shape(Mi, d, D.q_dim, h->n_sms, true, may_pair, &bn, &ks, &pr);
        ok = ok && launch_umma_gemm(h->m_attn, (bn == 256 && !pr) ? W.m_wo256 : W.m_wo, Mi, d, D.q_dim, bn, EPI_RESIDUAL, &re, nullptr,
                                    h->d_err, h->n_sms, s, ks, pr) == 0;
      }
    }
    timer.end();

    if (!small_rows) {
      timer.begin(PERCACHE_PH_NORM);
      launch_rmsnorm(h->resid, W.g_ffn, h->xn, Mi, d, D.rms_eps, s);
      timer.end();
    }

    SwigluEpilogue se{h->act, D.d_ffn};
    timer.begin(PERCACHE_PH_GATEUP);
    if (small_rows) {
      ok = ok && launch_small_gemm(EPI_SWIGLU, &se, Mi, 2 * D.d_ffn, d, h->resid, W.g_ffn, D.rms_eps, nullptr, W.wgu,
                                   h->gu_blk, h->n_sms, s) == 0;
    } else if (use_ref) {
      launch_ref_gemm(h->xn, W.wgu, h->cref, Mi, 2 * D.d_ffn, d, s);
      launch_ref_swiglu_epilogue(h->cref, Mi, D.d_ffn, h->gu_blk, se, s);
    } else {
      {
        int bn, ks, pr;
        umma_gemm_pick_shape(Mi, 2 * D.d_ffn, d, h->n_sms, false, may_pair, &bn, &ks, &pr);
        ok = ok && launch_umma_gemm(h->m_xn, (bn == 256 && !pr) ? W.m_wgu256 : W.m_wgu, Mi, 2 * D.d_ffn, d, bn, EPI_SWIGLU, &se, nullptr,
                                    h->d_err, h->n_sms, s, ks, pr) == 0;
      }
    }
    timer.end();

    timer.begin(PERCACHE_PH_DOWN);
    if (small_rows) {
      ok = ok && launch_small_gemm(EPI_RESIDUAL, &re, Mi, d, D.d_ffn, nullptr, nullptr, 0.f, h->act, W.wd, 0, h->n_sms,
                                   s) == 0;
    } else if (use_ref) {
      launch_ref_gemm(h->act, W.wd, h->cref, Mi, d, D.d_ffn, s);
      launch_ref_residual_epilogue(h->cref, Mi, d, re, s);
    } else {
      {
        int bn, ks, pr;
        umma_gemm_pick_shape(Mi, d, D.d_ffn, h->n_sms, true, may_pair, &bn, &ks, &pr);
        ok = ok && launch_umma_gemm(h->m_act, (bn == 256 && !pr) ? W.m_wd256 : W.m_wd, Mi, d, D.d_ffn, bn, EPI_RESIDUAL, &re, nullptr,
                                    h->d_err, h->n_sms, s, ks, pr) == 0;
      }
    }
    timer.end();
  }
  if (Mi > 0) capture(D.n_layers);
  return ok;
}


// ---------------------------------------------------------------------------------------------------------------
// Paper-faithful mode (PERCACHE_FLAG_PAPER_MODE): the scheme as the paper states it.  The chunk list is matched as a
// path of the cache tree (Section 3.2.2); a node holds the chunk's Q, K and V of every block, Q and K after position
// encoding (Sections 3.2.1, 5.3); all L_total rows of the prompt go through every block and only the rows of the
// matched chain (L_pre of them, less the dropped tail of its last node) skip the three projections and the position
// encoding (Appendix B.1).  Every row of the prompt owns a page slot (rows that are not chunk content, i.e. query
// tokens and a recomputed tail, get scratch pages for the duration of the call), the QKV epilogue writes pages only,
// and the attention reads Q, K and V through the prompt's page table: nothing is gathered or rotated.
// ---------------------------------------------------------------------------------------------------------------
int prefill_paper(percache* h, const percache_prompt_t* prompts, int32_t n_prompts, percache_result_t* results) {
  const auto t_host0 = std::chrono::steady_clock::now();
  const ModelDims& D = h->dims;
  const int d = D.d_model;
  if (h->flags & (PERCACHE_FLAG_REFERENCE_KERNELS | PERCACHE_FLAG_REFERENCE_ATTENTION)) return PERCACHE_E_INVAL;

  // ---------------------------------------------------------------- match the chains, sizes
  std::vector<std::vector<uint64_t>> keys(n_prompts);
  std::vector<std::vector<uint8_t>> hit(n_prompts);
  std::vector<int> n_match(n_prompts, 0), l_pre(n_prompts, 0);
  std::unordered_map<uint64_t, std::pair<int, int>> first_miss;
  std::unordered_map<uint64_t, int64_t> hit_uses;
  Plan plan;
  plan.cu_ctx.assign(1, 0);
  plan.cu_new.assign(1, 0);
  int64_t rows_total = 0, new_total = 0, hit_tokens = 0, pages_needed = 0, pt_entries = 0, visible_pairs = 0;
  int chunks_hit = 0, chunks_missed = 0;
  for (int b = 0; b < n_prompts; ++b) {
    const percache_prompt_t& P = prompts[b];
    if (P.n_chunks < 0 || P.n_query < 0 || (P.n_chunks > 0 && (!P.chunk_ids || !P.chunk_len)) ||
        (P.n_query > 0 && !P.query_hidden) || P.match_mode != PERCACHE_MATCH_PREFIX_PATH || P.reuse_tail_drop < 0 ||
        P.reuse_tail_drop % PAGE_TOKENS != 0)
      return PERCACHE_E_INVAL;
    keys[b].resize(static_cast<size_t>(P.n_chunks));
    hit[b].assign(static_cast<size_t>(P.n_chunks), 0);
    uint64_t path = PATH_KEY_SEED;
    bool walking = true;
    int64_t T = 0;
    for (int i = 0; i < P.n_chunks; ++i) {
      const int len = P.chunk_len[i];
      if (len <= 0 || len % PAGE_TOKENS != 0) return PERCACHE_E_INVAL;     // pages are copied whole in this mode
      if (!P.chunk_hidden || !P.chunk_hidden[i]) return PERCACHE_E_MISS_NO_INPUT;   // the whole prompt is embedded
      path = path_key_step(path, P.chunk_ids[i]);
      keys[b][i] = path;
      auto it = h->table.find(path);
      const bool stored = it != h->table.end();
      if (stored && it->second.n_tokens != len) return PERCACHE_E_LEN_MISMATCH;
      if (stored && walking) {
        hit[b][i] = 1;
        n_match[b] = i + 1;
        l_pre[b] += len;
        ++chunks_hit;
        ++hit_uses[path];
      } else {
        walking = false;
        ++chunks_missed;
        // the first prompt that computes a node keeps it; any other computation of it lives in scratch pages
        if (!stored && !first_miss.count(path)) first_miss.emplace(path, std::make_pair(b, i));
        pages_needed += len / PAGE_TOKENS;
      }
      T += len;
    }
    if (n_match[b] > 0) {
      if (P.reuse_tail_drop > P.chunk_len[n_match[b] - 1]) return PERCACHE_E_INVAL;
      l_pre[b] -= P.reuse_tail_drop;
      pages_needed += P.reuse_tail_drop / PAGE_TOKENS;
    }
    pages_needed += (P.n_query + PAGE_TOKENS - 1) / PAGE_TOKENS;
    T += P.n_query;
    if (T <= 0) return PERCACHE_E_INVAL;
    if (T > h->cfg.max_prompt_tokens) return PERCACHE_E_CAPACITY;
    if (results[b].out_capacity_rows < T || !results[b].out_hidden) return PERCACHE_E_CAPACITY;   // all rows come back
    hit_tokens += l_pre[b];
    rows_total += T;
    new_total += T - l_pre[b];
    pt_entries += (T + 127) / 128 * (128 / PAGE_TOKENS);
    if (rows_total > h->m_cap || rows_total > h->ctx_cap) return PERCACHE_E_CAPACITY;
    plan.cu_ctx.push_back(static_cast<int32_t>(rows_total));
    plan.cu_new.push_back(static_cast<int32_t>(new_total));
  }
  if (static_cast<size_t>(pt_entries) > 4 * static_cast<size_t>(h->ctx_cap)) return PERCACHE_E_CAPACITY;

  PageTxn txn(h);
  {
    std::vector<uint64_t> victims;
    const int rc = pick_victims(h, pages_needed, hit_uses, &victims);
    if (rc < 0) return rc;
    txn.set_victims(victims);
  }
  const int evicted = static_cast<int>(txn.victims.size());
  std::vector<std::pair<uint64_t, ChunkEntry>> pending;
  std::vector<int32_t> scratch;                   // pages that only live for this call
  auto fail = [&](int code) {
    if (txn.applied) h->plan = Plan();
    txn.undo();
    refresh_page_stats(h);
    return code;
  };

  // ---------------------------------------------------------------- index assembly
  const int64_t M = rows_total, M_new = new_total;
  int32_t* row_src = h->h_index;                  // new row -> row of the residual stream (its global row)
  int32_t* row_pos = row_src + h->m_cap;          // new row -> position
  int32_t* row_pool = row_pos + h->m_cap;         // new row -> page * 16 + offset
  int32_t* pos_all = row_pool + h->m_cap;         // global row -> position
  int32_t* page_table = pos_all + h->m_cap;       // in place of the gather items
  AttnItem* attn_items = reinterpret_cast<AttnItem*>(page_table + 4 * h->ctx_cap);
  int32_t* cta_first = reinterpret_cast<int32_t*>(attn_items) + 8 * h->max_attn_items;
  AttnMerge* merges = reinterpret_cast<AttnMerge*>(cta_first + h->n_sms + 1);
  struct Seg { const void* src; int on_device; int row0; int n; };
  std::vector<Seg> segs;
  std::vector<AttnBaseTile> base_tiles;
  plan.slot_chunk.resize(static_cast<size_t>(M));
  plan.slot_offset.resize(static_cast<size_t>(M));
  plan.slot_is_new.resize(static_cast<size_t>(M));
  plan.row_slot.resize(static_cast<size_t>(M_new));
  int64_t r = 0;
  int32_t pt_next = 0;
  for (int b = 0; b < n_prompts; ++b) {
    const percache_prompt_t& P = prompts[b];
    const int32_t g0 = plan.cu_ctx[b];
    const int32_t T = plan.cu_ctx[b + 1] - g0;
    const int32_t pt0 = pt_next;
    plan.ctx0.push_back(g0);
    plan.dec_len.push_back(0);
    int32_t t = 0;
    for (int i = 0; i <= P.n_chunks; ++i) {
      const bool is_query = (i == P.n_chunks);
      const int len = is_query ? P.n_query : P.chunk_len[i];
      if (len == 0) continue;
      const bool is_hit = !is_query && hit[b][i];
      const int reuse_len = !is_hit ? 0 : len - (i == n_match[b] - 1 ? P.reuse_tail_drop : 0);
      // pages of this stretch of slots: the stored node's, new ones that will become a node, or scratch
      std::vector<int32_t> fresh;
      const std::vector<int32_t>* stored_pages = nullptr;
      bool keep = false;
      if (is_hit) stored_pages = &h->table.find(keys[b][i])->second.pages;
      if (!is_query && !is_hit) {
        auto fm = first_miss.find(keys[b][i]);
        keep = fm != first_miss.end() && fm->second.first == b && fm->second.second == i;
      }
      const int n_fresh = (len - reuse_len + PAGE_TOKENS - 1) / PAGE_TOKENS;
      if (n_fresh > 0 && txn.take(n_fresh, &fresh) != PERCACHE_OK) return fail(PERCACHE_E_NOSPACE);
      if (keep) {
        ChunkEntry ent;
        ent.n_tokens = len;
        ent.serial = h->next_serial++;
        ent.pages = fresh;
        pending.emplace_back(keys[b][i], std::move(ent));
      } else {
        scratch.insert(scratch.end(), fresh.begin(), fresh.end());
      }
      for (int o = 0; o < len; o += PAGE_TOKENS)
        page_table[pt_next++] = o < reuse_len ? (*stored_pages)[o / PAGE_TOKENS] : fresh[(o - reuse_len) / PAGE_TOKENS];
      segs.push_back(Seg{is_query ? P.query_hidden : P.chunk_hidden[i], P.hidden_on_device, g0 + t, len});
      for (int o = 0; o < len; ++o) {
        plan.slot_chunk[g0 + t + o] = i;
        plan.slot_offset[g0 + t + o] = o;
        plan.slot_is_new[g0 + t + o] = o < reuse_len ? 0 : 1;
        pos_all[g0 + t + o] = t + o;
        visible_pairs += t + o + 1;
        if (o >= reuse_len) {
          row_src[r] = g0 + t + o;
          row_pos[r] = t + o;
          row_pool[r] = fresh[(o - reuse_len) / PAGE_TOKENS] * PAGE_TOKENS + ((o - reuse_len) % PAGE_TOKENS);
          plan.row_slot[r] = t + o;
          ++r;
        }
      }
      t += len;
    }
    // pad the prompt's table to whole 128-slot blocks with its last page (those slots are never visible)
    const int32_t last_page = page_table[pt_next - 1];
    while ((pt_next - pt0) % (128 / PAGE_TOKENS) != 0) page_table[pt_next++] = last_page;
    for (int32_t r0 = 0; r0 < T; r0 += 128) {
      AttnBaseTile a{};
      a.row0 = g0 + r0;
      a.n_rows = std::min(128, T - r0);
      a.ctx0 = pt0;                                   // the paged attention reads ctx0 as the table offset
      a.n_blocks = (r0 + a.n_rows + 127) / 128;
      base_tiles.push_back(a);
    }
  }
  int n_attn_ctas = 0, n_merges = 0;
  {
    std::vector<AttnItem> v_items;
    std::vector<int32_t> v_first;
    std::vector<AttnMerge> v_merges;
    plan_attention(base_tiles, D.n_kv_heads * (D.n_q_heads / D.n_kv_heads / 2), h->n_sms, h->partial_slots, &v_items,
                   &v_first, &v_merges);
    if (v_items.size() > h->max_attn_items || v_merges.size() > h->max_attn_merges ||
        v_first.size() > static_cast<size_t>(h->n_sms) + 1)
      return fail(PERCACHE_E_CAPACITY);
    std::copy(v_items.begin(), v_items.end(), attn_items);
    std::fill(cta_first, cta_first + h->n_sms + 1, static_cast<int32_t>(v_items.size()));
    std::copy(v_first.begin(), v_first.end(), cta_first);
    std::copy(v_merges.begin(), v_merges.end(), merges);
    n_attn_ctas = static_cast<int>(v_first.size()) - 1;
    n_merges = static_cast<int>(v_merges.size());
  }
  const double plan_us =
      std::chrono::duration<double, std::micro>(std::chrono::steady_clock::now() - t_host0).count();

  // ---------------------------------------------------------------- device work
  cudaStream_t s = h->stream;
  percache_stats_t& st = h->stats;
  std::memset(st.phase_us, 0, sizeof(st.phase_us));
  std::memset(st.phase_launches, 0, sizeof(st.phase_launches));
  PhaseTimer timer(h);
  bool ok = true;
  txn.apply();
  const size_t used_ints = static_cast<size_t>(reinterpret_cast<int32_t*>(merges + n_merges) - h->h_index);
  ok = ok && cudaMemcpyAsync(h->d_index, h->h_index, used_ints * sizeof(int32_t), cudaMemcpyHostToDevice, s) == cudaSuccess;
  ok = ok && cudaMemsetAsync(h->d_err, 0, sizeof(int), s) == cudaSuccess;
  const DevIndex ix = dev_index(h);
  const int32_t* d_page_table = reinterpret_cast<const int32_t*>(ix.items);
  timer.begin(PERCACHE_PH_IO);
  for (const Seg& sg : segs)
    ok = ok && cudaMemcpyAsync(h->xin + static_cast<size_t>(sg.row0) * d, sg.src, static_cast<size_t>(sg.n) * d * 2,
                               sg.on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice, s) == cudaSuccess;
  cudaEventRecord(h->ev_begin, s);
  launch_bf16_to_f32(h->xin, h->resid, M * d, s);
  timer.end();

  const int Mi = static_cast<int>(M), Mn = static_cast<int>(M_new);
  const size_t pool_layer = static_cast<size_t>(h->cfg.pool_pages) * PAGE_TOKENS;
  const bool may_pair = !(h->flags & PERCACHE_FLAG_SINGLE_CTA_GEMM);
  auto gemm = [&](const GemmOperand& A, const GemmOperand& B128, const GemmOperand& B256, int rows, int N, int K,
                  GemmEpilogueKind kind, const void* epi, bool residual) {
    int bn, ks, pr;
    umma_gemm_pick_shape(rows, N, K, h->n_sms, residual, may_pair, &bn, &ks, &pr);
    return launch_umma_gemm(A, (bn == 256 && !pr) ? B256 : B128, rows, N, K, bn, kind, epi, nullptr, h->d_err, h->n_sms, s,
                            ks, pr) == 0;
  };
  for (int l = 0; l < D.n_layers && ok; ++l) {
    LayerWeights& W = h->layers[l];
    if (Mn > 0) {       // projections and position encoding on the rows the loaded tensors do not cover
      timer.begin(PERCACHE_PH_NORM);
      launch_rmsnorm(h->resid, W.g_attn, h->xn, Mn, d, D.rms_eps, s, ix.row_slot);
      timer.end();
      QkvEpilogue qe{};
      qe.rows = RowIndex{ix.row_slot, ix.row_pos, ix.row_pool};
      qe.rope = h->rope;
      qe.qpool = h->qpool + l * pool_layer * D.q_dim;
      qe.kpool = h->kpool + l * pool_layer * D.kv_dim;
      qe.vpool = h->vpool + l * pool_layer * D.kv_dim;
      qe.n_q_heads = D.n_q_heads;
      qe.n_kv_heads = D.n_kv_heads;
      qe.paged = 1;
      timer.begin(PERCACHE_PH_QKV);
      ok = ok && gemm(h->m_xn, W.m_wqkv, W.m_wqkv256, Mn, D.qkv_dim, d, EPI_QKV, &qe, false);
      timer.end();
    }
    // loaded and computed tensors side by side in the pages: the sequence is L_total rows long again
    timer.begin(PERCACHE_PH_ATTN);
    ok = ok && launch_umma_attention(W.paged_maps, ix.attn_items, ix.cta_first, n_attn_ctas, ix.row_ctx0, h->attn_out,
                                     h->partial_o, h->partial_ml, D.n_q_heads, D.n_kv_heads, h->d_err, s,
                                     d_page_table, 1) == 0;
    launch_attention_merge(ix.merges, n_merges, h->partial_o, h->partial_ml, h->attn_out, D.n_q_heads, D.n_kv_heads, s);
    timer.end();
    ResidualEpilogue re{h->resid, d};
    timer.begin(PERCACHE_PH_OPROJ);
    ok = ok && gemm(h->m_attn, W.m_wo, W.m_wo256, Mi, d, D.q_dim, EPI_RESIDUAL, &re, true);
    timer.end();
    timer.begin(PERCACHE_PH_NORM);
    launch_rmsnorm(h->resid, W.g_ffn, h->xn, Mi, d, D.rms_eps, s);
    timer.end();
    SwigluEpilogue se{h->act, D.d_ffn};
    timer.begin(PERCACHE_PH_GATEUP);
    ok = ok && gemm(h->m_xn, W.m_wgu, W.m_wgu256, Mi, 2 * D.d_ffn, d, EPI_SWIGLU, &se, false);
    timer.end();
    timer.begin(PERCACHE_PH_DOWN);
    ok = ok && gemm(h->m_act, W.m_wd, W.m_wd256, Mi, d, D.d_ffn, EPI_RESIDUAL, &re, true);
    timer.end();
  }
  cudaEventRecord(h->ev_end, s);
  timer.begin(PERCACHE_PH_IO);
  for (int b = 0; b < n_prompts && ok; ++b) {
    const int T = plan.cu_ctx[b + 1] - plan.cu_ctx[b];
    ok = ok && cudaMemcpyAsync(results[b].out_hidden, h->resid + static_cast<size_t>(plan.cu_ctx[b]) * d,
                               static_cast<size_t>(T) * d * sizeof(float),
                               results[b].out_on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyDeviceToHost, s) == cudaSuccess;
  }
  ok = ok && cudaMemcpyAsync(h->h_err, h->d_err, sizeof(int), cudaMemcpyDeviceToHost, s) == cudaSuccess;
  timer.end();
  const cudaError_t sync_rc = cudaStreamSynchronize(s);
  if (!ok || sync_rc != cudaSuccess || cudaGetLastError() != cudaSuccess) return fail(PERCACHE_E_CUDA);
  if (*h->h_err != 0) return fail(PERCACHE_E_DEVICE_TIMEOUT);

  // ---------------------------------------------------------------- commit
  for (auto& pe : pending) h->table.emplace(pe.first, std::move(pe.second));
  for (const auto& hu : hit_uses) h->table[hu.first].retrievals += hu.second;
  release_pages(h, scratch);
  st.evictions = evicted;
  for (int b = 0; b < n_prompts; ++b) {
    results[b].n_total = plan.cu_ctx[b + 1] - plan.cu_ctx[b];
    results[b].n_new = plan.cu_new[b + 1] - plan.cu_new[b];
    if (results[b].hit_mask && prompts[b].n_chunks > 0)
      std::memcpy(results[b].hit_mask, hit[b].data(), static_cast<size_t>(prompts[b].n_chunks));
  }
  h->plan = std::move(plan);
  st.n_prompts = n_prompts;
  st.chunks_hit = chunks_hit;
  st.chunks_missed = chunks_missed;
  st.ctx_tokens = rows_total;
  st.hit_tokens = hit_tokens;
  st.new_rows = new_total;
  refresh_page_stats(h);
  st.host_plan_us = plan_us;
  st.attn_visible_pairs = visible_pairs;
  st.gather_free = 1;            // this mode never gathers
  float ms = 0.f;
  cudaEventElapsedTime(&ms, h->ev_begin, h->ev_end);
  st.device_us = 1000.0 * ms;
  timer.collect();
  return PERCACHE_OK;
}


}  // namespace

extern "C" {

const char* percache_strerror(int code) {
  switch (code) {
    case PERCACHE_OK: return "ok";
    case PERCACHE_E_INVAL: return "invalid argument";
    case PERCACHE_E_NOMEM: return "out of memory";
    case PERCACHE_E_NOSPACE: return "paged store is full";
    case PERCACHE_E_EXISTS: return "chunk id already stored";
    case PERCACHE_E_LEN_MISMATCH: return "chunk stored with a different length";
    case PERCACHE_E_MISS_NO_INPUT: return "chunk not stored and no hidden states given";
    case PERCACHE_E_CAPACITY: return "capacity fixed at creation exceeded";
    case PERCACHE_E_DEVICE_TIMEOUT: return "bounded wait inside a kernel ran out";
    case PERCACHE_E_CUDA: return "CUDA call failed";
    case PERCACHE_E_NOTFOUND: return "chunk id not stored";
    default: return "unknown error";
  }
}

int percache_create(const percache_config_t* cfg, const percache_layer_weights_t* lw, int32_t weights_on_device,
                    percache_t** out) {
  if (!cfg || !lw || !out) return PERCACHE_E_INVAL;
  *out = nullptr;
  if (cfg->n_layers <= 0 || cfg->n_layers > 64 || cfg->head_dim != HEAD_DIM || cfg->page_tokens != PAGE_TOKENS ||
      cfg->d_model <= 0 || cfg->d_model % 128 != 0 || cfg->d_ffn <= 0 || cfg->d_ffn % 64 != 0 ||
      cfg->n_kv_heads <= 0 || cfg->n_q_heads <= 0 || cfg->n_q_heads % (2 * cfg->n_kv_heads) != 0 ||
      cfg->pool_pages <= 0 || cfg->max_prompt_tokens <= 0 || cfg->max_batch_prompts <= 0 ||
      cfg->max_batch_ctx_tokens <= 0 || cfg->max_batch_new_rows <= 0 || cfg->pool_pages > (INT32_MAX / PAGE_TOKENS) ||
      cfg->max_batch_ctx_tokens > INT32_MAX / 2 || cfg->max_batch_new_rows > INT32_MAX / 2)
    return PERCACHE_E_INVAL;
  for (int l = 0; l < cfg->n_layers; ++l) {
    const percache_layer_weights_t& S = lw[l];
    if (!S.attn_norm || !S.wq || !S.wk || !S.wv || !S.wo || !S.ffn_norm || !S.w_gate || !S.w_up || !S.w_down)
      return PERCACHE_E_INVAL;
  }
  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || cfg->device < 0 || cfg->device >= n_dev) {
    cudaGetLastError();
    return PERCACHE_E_CUDA;
  }
  if (cudaSetDevice(cfg->device) != cudaSuccess) return PERCACHE_E_CUDA;
  if (init_driver_api() != 0) return PERCACHE_E_CUDA;

  percache* h = new (std::nothrow) percache();
  if (!h) return PERCACHE_E_NOMEM;
  h->cfg = *cfg;
  h->stream = static_cast<cudaStream_t>(cfg->stream);
  h->flags = cfg->flags;
  ModelDims& D = h->dims;
  D.n_layers = cfg->n_layers; D.d_model = cfg->d_model; D.n_q_heads = cfg->n_q_heads; D.n_kv_heads = cfg->n_kv_heads;
  D.d_ffn = cfg->d_ffn; D.q_dim = cfg->n_q_heads * HEAD_DIM; D.kv_dim = cfg->n_kv_heads * HEAD_DIM;
  D.qkv_dim = D.q_dim + 2 * D.kv_dim; D.rms_eps = cfg->rms_eps;
  h->m_cap = cfg->max_batch_new_rows;
  h->ctx_cap = cfg->max_batch_ctx_tokens;
  cudaDeviceGetAttribute(&h->n_sms, cudaDevAttrMultiProcessorCount, cfg->device);
  h->gu_blk = UMMA_GEMM_MIN_BLOCK_N / 2;

  const int L = D.n_layers, d = D.d_model, F = D.d_ffn;
  bool ok = true;
  const size_t pool_elems = static_cast<size_t>(L) * cfg->pool_pages * PAGE_TOKENS * D.kv_dim;
  const size_t ctx_elems = static_cast<size_t>(L) * h->ctx_cap * D.kv_dim;
  ok = ok && dev_alloc(h, &h->kpool, pool_elems) && dev_alloc(h, &h->vpool, pool_elems);
  h->paper_mode = (cfg->flags & PERCACHE_FLAG_PAPER_MODE) != 0;
  const size_t qpool_elems = static_cast<size_t>(L) * cfg->pool_pages * PAGE_TOKENS * D.q_dim;
  if (h->paper_mode) ok = ok && dev_alloc(h, &h->qpool, qpool_elems);
  ok = ok && dev_alloc(h, &h->kctx, ctx_elems) && dev_alloc(h, &h->vctx, ctx_elems);
  ok = ok && dev_alloc(h, &h->rope, static_cast<size_t>(cfg->max_prompt_tokens) * ROPE_HALF);
  ok = ok && dev_alloc(h, &h->resid, static_cast<size_t>(h->m_cap) * d);
  ok = ok && dev_alloc(h, &h->xin, static_cast<size_t>(h->m_cap) * d);
  ok = ok && dev_alloc(h, &h->xn, static_cast<size_t>(h->m_cap) * d);
  ok = ok && dev_alloc(h, &h->qbuf, static_cast<size_t>(h->m_cap) * D.q_dim);
  ok = ok && dev_alloc(h, &h->attn_out, static_cast<size_t>(h->m_cap) * D.q_dim);
  ok = ok && dev_alloc(h, &h->act, static_cast<size_t>(h->m_cap) * F);
  ok = ok && dev_alloc(h, &h->d_err, 1);
  // index block: 4 row arrays + gather items (worst case one per context token) + attention tiles
  // (an attention item per unit of every tile, plus the parts the scheduler cuts: at most two per CTA)
  const size_t max_tiles = static_cast<size_t>(h->m_cap / 128 + cfg->max_batch_prompts + 2);
  const size_t units_per_tile = static_cast<size_t>(D.n_kv_heads) * (D.n_q_heads / D.n_kv_heads / 2);
  h->partial_slots = 2 * h->n_sms + 2;
  h->max_attn_items = max_tiles * units_per_tile + 2 * static_cast<size_t>(h->n_sms);
  h->max_attn_merges = std::max(static_cast<size_t>(h->n_sms) + 1,      // prefill: at most one cut unit per CTA
                                static_cast<size_t>(cfg->max_batch_prompts) * D.n_kv_heads);   // decode: (prompt, KV head)
  h->index_ints = 4 * static_cast<size_t>(h->m_cap) + 4 * static_cast<size_t>(h->ctx_cap) + 8 * h->max_attn_items +
                  static_cast<size_t>(h->n_sms) + 1 + 8 * h->max_attn_merges;
  ok = ok && dev_alloc(h, &h->partial_o, static_cast<size_t>(h->partial_slots) * 2 * 128 * HEAD_DIM);
  ok = ok && dev_alloc(h, &h->partial_ml, static_cast<size_t>(h->partial_slots) * 2 * 128 * 2);
  ok = ok && dev_alloc(h, &h->d_index, h->index_ints);
  if (ok && cudaMallocHost(reinterpret_cast<void**>(&h->h_index), h->index_ints * sizeof(int32_t)) != cudaSuccess) ok = false;
  if (ok && cudaMallocHost(reinterpret_cast<void**>(&h->h_err), sizeof(int)) != cudaSuccess) ok = false;
  h->layers.resize(L);
  for (int l = 0; ok && l < L; ++l) {
    LayerWeights& W = h->layers[l];
    ok = ok && dev_alloc(h, &W.wqkv, static_cast<size_t>(D.qkv_dim) * d) && dev_alloc(h, &W.wo, static_cast<size_t>(d) * D.q_dim) &&
         dev_alloc(h, &W.wgu, static_cast<size_t>(2 * F) * d) && dev_alloc(h, &W.wd, static_cast<size_t>(d) * F) &&
         dev_alloc(h, &W.g_attn, d) && dev_alloc(h, &W.g_ffn, d);
  }
  if (!ok) {
    cudaGetLastError();
    destroy_impl(h);
    return PERCACHE_E_NOMEM;
  }
  if (cudaEventCreate(&h->ev_begin) != cudaSuccess || cudaEventCreate(&h->ev_end) != cudaSuccess) {
    destroy_impl(h);
    return PERCACHE_E_CUDA;
  }
  h->events.assign(MAX_EVENTS, nullptr);
  for (auto& e : h->events)
    if (cudaEventCreate(&e) != cudaSuccess) { destroy_impl(h); return PERCACHE_E_CUDA; }
  if (cudaStreamCreateWithFlags(&h->side, cudaStreamNonBlocking) != cudaSuccess ||
      cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming) != cudaSuccess) {
    destroy_impl(h);
    return PERCACHE_E_CUDA;
  }
  h->ev_gather.assign(D.n_layers, nullptr);
  for (auto& e : h->ev_gather)
    if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) { destroy_impl(h); return PERCACHE_E_CUDA; }

  // Operand buffers start as zeros: rows and context slots a call does not write are still read by
  // whole-tile TMA loads (and then masked or never stored), so they must never hold NaN bit patterns.
  cudaMemsetAsync(h->kctx, 0, ctx_elems * 2, h->stream);
  cudaMemsetAsync(h->vctx, 0, ctx_elems * 2, h->stream);
  cudaMemsetAsync(h->qbuf, 0, static_cast<size_t>(h->m_cap) * D.q_dim * 2, h->stream);
  cudaMemsetAsync(h->attn_out, 0, static_cast<size_t>(h->m_cap) * D.q_dim * 2, h->stream);
  cudaMemsetAsync(h->xn, 0, static_cast<size_t>(h->m_cap) * d * 2, h->stream);
  cudaMemsetAsync(h->act, 0, static_cast<size_t>(h->m_cap) * F * 2, h->stream);
  // the paged forms of the attention copy whole pages, also ones a prompt only partly fills
  if (h->paper_mode) cudaMemsetAsync(h->qpool, 0, qpool_elems * 2, h->stream);
  cudaMemsetAsync(h->kpool, 0, pool_elems * 2, h->stream);
  cudaMemsetAsync(h->vpool, 0, pool_elems * 2, h->stream);

  // ---- weights: bf16 -> fp16 copies in the layouts the GEMMs read.  Every bf16 value of magnitude
  // >= 2^-17 is exactly representable in fp16; smaller ones round with absolute error <= 2^-25.
  cudaStream_t s = h->stream;
  __nv_bfloat16 *tmp0 = nullptr, *tmp1 = nullptr;
  const size_t max_w = std::max<size_t>(static_cast<size_t>(F) * d, static_cast<size_t>(D.q_dim) * d);
  bool cuda_ok = true;
  if (!weights_on_device) {
    if (cudaMalloc(reinterpret_cast<void**>(&tmp0), max_w * 2) != cudaSuccess ||
        cudaMalloc(reinterpret_cast<void**>(&tmp1), max_w * 2) != cudaSuccess) {
      cudaGetLastError();
      if (tmp0) cudaFree(tmp0);
      destroy_impl(h);
      return PERCACHE_E_NOMEM;
    }
  }
  const size_t ctx_layer = static_cast<size_t>(h->ctx_cap) * D.kv_dim;
  for (int l = 0; l < L && cuda_ok; ++l) {
    LayerWeights& W = h->layers[l];
    const percache_layer_weights_t& S = lw[l];
    const __nv_bfloat16* p;
    // stream order keeps each conversion ahead of the next copy into the same staging buffer
    p = stage_bf16(S.wq, static_cast<size_t>(D.q_dim) * d, weights_on_device, tmp0, s, &cuda_ok);
    launch_bf16_to_f16(p, W.wqkv, static_cast<int64_t>(D.q_dim) * d, s);
    p = stage_bf16(S.wk, static_cast<size_t>(D.kv_dim) * d, weights_on_device, tmp1, s, &cuda_ok);
    launch_bf16_to_f16(p, W.wqkv + static_cast<size_t>(D.q_dim) * d, static_cast<int64_t>(D.kv_dim) * d, s);
    p = stage_bf16(S.wv, static_cast<size_t>(D.kv_dim) * d, weights_on_device, tmp0, s, &cuda_ok);
    launch_bf16_to_f16(p, W.wqkv + static_cast<size_t>(D.q_dim + D.kv_dim) * d, static_cast<int64_t>(D.kv_dim) * d, s);
    p = stage_bf16(S.wo, static_cast<size_t>(d) * D.q_dim, weights_on_device, tmp1, s, &cuda_ok);
    launch_bf16_to_f16(p, W.wo, static_cast<int64_t>(d) * D.q_dim, s);
    const __nv_bfloat16* pg = stage_bf16(S.w_gate, static_cast<size_t>(F) * d, weights_on_device, tmp0, s, &cuda_ok);
    const __nv_bfloat16* pu = stage_bf16(S.w_up, static_cast<size_t>(F) * d, weights_on_device, tmp1, s, &cuda_ok);
    launch_interleave_rows_bf16_to_f16(pg, pu, W.wgu, F, d, h->gu_blk, s);
    p = stage_bf16(S.w_down, static_cast<size_t>(d) * F, weights_on_device, tmp0, s, &cuda_ok);
    launch_bf16_to_f16(p, W.wd, static_cast<int64_t>(d) * F, s);
    p = stage_bf16(S.attn_norm, d, weights_on_device, tmp1, s, &cuda_ok);
    launch_bf16_to_f32(p, W.g_attn, d, s);
    p = stage_bf16(S.ffn_norm, d, weights_on_device, tmp0, s, &cuda_ok);
    launch_bf16_to_f32(p, W.g_ffn, d, s);
    const int bn = UMMA_GEMM_MIN_BLOCK_N;
    cuda_ok = cuda_ok && make_operand_map(&W.m_wqkv, W.wqkv, D.qkv_dim, d, bn) == 0 &&
              make_operand_map(&W.m_wo, W.wo, d, D.q_dim, bn) == 0 &&
              make_operand_map(&W.m_wgu, W.wgu, 2 * F, d, bn) == 0 && make_operand_map(&W.m_wd, W.wd, d, F, bn) == 0;
    cuda_ok = cuda_ok && make_operand_map(&W.m_wqkv256, W.wqkv, D.qkv_dim, d, 256) == 0 &&
              make_operand_map(&W.m_wo256, W.wo, d, D.q_dim, 256) == 0 &&
              make_operand_map(&W.m_wgu256, W.wgu, 2 * F, d, 256) == 0 && make_operand_map(&W.m_wd256, W.wd, d, F, 256) == 0;
    cuda_ok = cuda_ok && make_attn_maps(&W.attn_maps, h->qbuf, h->m_cap, D.q_dim, h->kctx + l * ctx_layer,
                                        h->vctx + l * ctx_layer, h->ctx_cap, D.kv_dim) == 0;
    {
      // gather-free form of the default mode: Q as above, K and V one page (16 rows) of a 64-column half per copy
      const size_t pl = static_cast<size_t>(cfg->pool_pages) * PAGE_TOKENS;
      W.gf_maps = W.attn_maps;
      const uint32_t box[2] = {64u, static_cast<uint32_t>(PAGE_TOKENS)};
      const uint64_t vd[2] = {static_cast<uint64_t>(D.kv_dim), static_cast<uint64_t>(pl)};
      const uint64_t vs[1] = {static_cast<uint64_t>(D.kv_dim) * 2};
      cuda_ok = cuda_ok && encode_f16_map(&W.gf_maps.v, h->vpool + l * pl * D.kv_dim, 2, vd, vs, box) == 0 &&
                encode_f16_map(&W.gf_maps.k, h->kpool + l * pl * D.kv_dim, 2, vd, vs, box) == 0;
    }
    if (h->paper_mode) {
      const size_t pl = static_cast<size_t>(cfg->pool_pages) * PAGE_TOKENS;
      cuda_ok = cuda_ok && make_paged_attn_maps(&W.paged_maps, h->qpool + l * pl * D.q_dim, h->kpool + l * pl * D.kv_dim,
                                                h->vpool + l * pl * D.kv_dim, cfg->pool_pages, D.q_dim, D.kv_dim) == 0;
    }
  }
  launch_build_rope_table(h->rope, cfg->max_prompt_tokens, static_cast<double>(cfg->rope_theta), s);
  cuda_ok = cuda_ok && make_operand_map(&h->m_xn, h->xn, h->m_cap, d, 128) == 0 &&
            make_operand_map(&h->m_attn, h->attn_out, h->m_cap, D.q_dim, 128) == 0 &&
            make_operand_map(&h->m_act, h->act, h->m_cap, F, 128) == 0;
  if (cudaStreamSynchronize(s) != cudaSuccess) cuda_ok = false;
  if (tmp0) cudaFree(tmp0);
  if (tmp1) cudaFree(tmp1);
  if (!cuda_ok || cudaGetLastError() != cudaSuccess) {
    destroy_impl(h);
    return PERCACHE_E_CUDA;
  }
  h->free_pages.resize(static_cast<size_t>(cfg->pool_pages));
  for (int64_t i = 0; i < cfg->pool_pages; ++i)
    h->free_pages[static_cast<size_t>(i)] = static_cast<int32_t>(cfg->pool_pages - 1 - i);   // pops give 0, 1, 2, ...
  h->store_limit = cfg->pool_pages;
  refresh_page_stats(h);
  *out = h;
  return PERCACHE_OK;
}

int percache_set_store_limit(percache_t* h, int64_t pages) {
  if (!h || pages < 1 || pages > h->cfg.pool_pages) return PERCACHE_E_INVAL;
  const int64_t old = h->store_limit;
  h->store_limit = pages;
  std::vector<uint64_t> victims;
  const int rc = pick_victims(h, 0, {}, &victims);
  if (rc < 0) { h->store_limit = old; return rc; }
  for (uint64_t id : victims) {
    auto it = h->table.find(id);
    release_pages(h, it->second.pages);
    h->table.erase(it);
  }
  h->stats.evictions = rc;
  refresh_page_stats(h);
  return PERCACHE_OK;
}

int percache_chunk_info(percache_t* h, uint64_t chunk_id, int32_t* n_tokens, int64_t* retrievals) {
  if (!h) return PERCACHE_E_INVAL;
  auto it = h->table.find(chunk_id);
  if (it == h->table.end()) return PERCACHE_E_NOTFOUND;
  if (n_tokens) *n_tokens = it->second.n_tokens;
  if (retrievals) *retrievals = it->second.retrievals;
  return PERCACHE_OK;
}

uint64_t percache_path_key(const uint64_t* chunk_ids, int32_t n) {
  uint64_t path = PATH_KEY_SEED;
  for (int32_t i = 0; chunk_ids && i < n; ++i) path = path_key_step(path, chunk_ids[i]);
  return path;
}

int percache_destroy(percache_t* h) {
  destroy_impl(h);
  return PERCACHE_OK;
}

int percache_set_flags(percache_t* h, uint32_t flags) {
  if (!h) return PERCACHE_E_INVAL;
  h->flags = (flags & ~PERCACHE_FLAG_PAPER_MODE) | (h->flags & PERCACHE_FLAG_PAPER_MODE);   // the mode is fixed at creation
  return PERCACHE_OK;
}

int percache_has_chunk(percache_t* h, uint64_t chunk_id, int32_t* n_tokens) {
  if (!h) return PERCACHE_E_INVAL;
  auto it = h->table.find(chunk_id);
  if (it == h->table.end()) return PERCACHE_E_NOTFOUND;
  if (n_tokens) *n_tokens = it->second.n_tokens;
  return PERCACHE_OK;
}

int percache_drop_chunk(percache_t* h, uint64_t chunk_id) {
  if (!h) return PERCACHE_E_INVAL;
  auto it = h->table.find(chunk_id);
  if (it == h->table.end()) return PERCACHE_E_NOTFOUND;
  release_pages(h, it->second.pages);
  h->table.erase(it);
  refresh_page_stats(h);
  return PERCACHE_OK;
}

int percache_put_chunk_kv(percache_t* h, uint64_t chunk_id, int32_t n_tokens, const void* k, const void* v,
                          int32_t ptr_is_device) {
  if (!h || !k || !v || n_tokens <= 0 || h->paper_mode) return PERCACHE_E_INVAL;   // that mode's entries hold Q as well
  if (cudaSetDevice(h->cfg.device) != cudaSuccess) return PERCACHE_E_CUDA;
  if (h->table.count(chunk_id)) return PERCACHE_E_EXISTS;
  const int n_pages = (n_tokens + PAGE_TOKENS - 1) / PAGE_TOKENS;
  ChunkEntry ent;
  ent.n_tokens = n_tokens;
  std::vector<uint64_t> victims;
  int rc = pick_victims(h, n_pages, {}, &victims);
  if (rc < 0) return rc;
  const int evicted = rc;
  rc = PERCACHE_OK;
  const size_t elems = static_cast<size_t>(h->dims.n_layers) * n_tokens * h->dims.kv_dim;
  __nv_bfloat16 *dk = nullptr, *dv = nullptr;
  if (!ptr_is_device) {      // staging copies first: an allocation failure must leave the store untouched
    if (cudaMalloc(reinterpret_cast<void**>(&dk), elems * 2) != cudaSuccess ||
        cudaMalloc(reinterpret_cast<void**>(&dv), elems * 2) != cudaSuccess) {
      cudaGetLastError();
      if (dk) cudaFree(dk);
      return PERCACHE_E_NOMEM;
    }
    if (cudaMemcpyAsync(dk, k, elems * 2, cudaMemcpyHostToDevice, h->stream) != cudaSuccess ||
        cudaMemcpyAsync(dv, v, elems * 2, cudaMemcpyHostToDevice, h->stream) != cudaSuccess)
      rc = PERCACHE_E_CUDA;
  } else {
    dk = static_cast<__nv_bfloat16*>(const_cast<void*>(k));
    dv = static_cast<__nv_bfloat16*>(const_cast<void*>(v));
  }
  PageTxn txn(h);
  if (rc == PERCACHE_OK) {
    txn.set_victims(victims);
    rc = txn.take(n_pages, &ent.pages);
  }
  if (rc == PERCACHE_OK) {
    txn.apply();
    ent.serial = h->next_serial++;
    rc = with_chunk_pages(h, ent.pages, [&](const int32_t* d_pages) {
      launch_chunk_pages_copy(dk, h->kpool, d_pages, n_tokens, h->dims.n_layers, h->cfg.pool_pages, h->dims.kv_dim, 1,
                              h->stream);
      launch_chunk_pages_copy(dv, h->vpool, d_pages, n_tokens, h->dims.n_layers, h->cfg.pool_pages, h->dims.kv_dim, 1,
                              h->stream);
    });
  }
  if (!ptr_is_device) {
    cudaStreamSynchronize(h->stream);
    cudaFree(dk);
    cudaFree(dv);
  }
  if (rc != PERCACHE_OK) { txn.undo(); refresh_page_stats(h); return rc; }
  h->stats.evictions = evicted;
  h->table.emplace(chunk_id, std::move(ent));
  refresh_page_stats(h);
  return PERCACHE_OK;
}

int percache_put_chunk_synthetic(percache_t* h, uint64_t chunk_id, int32_t n_tokens, uint64_t seed) {
  if (!h || n_tokens <= 0 || h->paper_mode) return PERCACHE_E_INVAL;
  if (cudaSetDevice(h->cfg.device) != cudaSuccess) return PERCACHE_E_CUDA;
  if (h->table.count(chunk_id)) return PERCACHE_E_EXISTS;
  ChunkEntry ent;
  ent.n_tokens = n_tokens;
  const int n_pages = (n_tokens + PAGE_TOKENS - 1) / PAGE_TOKENS;
  std::vector<uint64_t> victims;
  int rc = pick_victims(h, n_pages, {}, &victims);
  if (rc < 0) return rc;
  const int evicted = rc;
  PageTxn txn(h);
  txn.set_victims(victims);
  rc = txn.take(n_pages, &ent.pages);
  if (rc != PERCACHE_OK) { txn.undo(); return rc; }
  txn.apply();
  ent.serial = h->next_serial++;
  rc = with_chunk_pages(h, ent.pages, [&](const int32_t* d_pages) {
    launch_fill_synthetic(h->kpool, h->vpool, d_pages, n_tokens, h->dims.n_layers, h->cfg.pool_pages, h->dims.kv_dim,
                          seed, chunk_id, h->stream);
  });
  if (rc != PERCACHE_OK) { txn.undo(); refresh_page_stats(h); return rc; }
  h->stats.evictions = evicted;
  h->table.emplace(chunk_id, std::move(ent));
  refresh_page_stats(h);
  return PERCACHE_OK;
}

int percache_get_chunk_kv(percache_t* h, uint64_t chunk_id, void* k_host, void* v_host) {
  if (!h || !k_host || !v_host) return PERCACHE_E_INVAL;
  if (cudaSetDevice(h->cfg.device) != cudaSuccess) return PERCACHE_E_CUDA;
  auto it = h->table.find(chunk_id);
  if (it == h->table.end()) return PERCACHE_E_NOTFOUND;
  const ChunkEntry& ent = it->second;
  const size_t elems = static_cast<size_t>(h->dims.n_layers) * ent.n_tokens * h->dims.kv_dim;
  __nv_bfloat16 *dk = nullptr, *dv = nullptr;
  if (cudaMalloc(reinterpret_cast<void**>(&dk), elems * 2) != cudaSuccess ||
      cudaMalloc(reinterpret_cast<void**>(&dv), elems * 2) != cudaSuccess) {
    cudaGetLastError();
    if (dk) cudaFree(dk);
    return PERCACHE_E_NOMEM;
  }
  int rc = with_chunk_pages(h, ent.pages, [&](const int32_t* d_pages) {
    launch_chunk_pages_copy(dk, h->kpool, d_pages, ent.n_tokens, h->dims.n_layers, h->cfg.pool_pages, h->dims.kv_dim, 0,
                            h->stream);
    launch_chunk_pages_copy(dv, h->vpool, d_pages, ent.n_tokens, h->dims.n_layers, h->cfg.pool_pages, h->dims.kv_dim, 0,
                            h->stream);
  });
  if (rc == PERCACHE_OK && (cudaMemcpy(k_host, dk, elems * 2, cudaMemcpyDeviceToHost) != cudaSuccess ||
                            cudaMemcpy(v_host, dv, elems * 2, cudaMemcpyDeviceToHost) != cudaSuccess))
    rc = PERCACHE_E_CUDA;
  cudaFree(dk);
  cudaFree(dv);
  return rc;
}

int percache_get_chunk_q(percache_t* h, uint64_t chunk_id, void* q_host) {
  if (!h || !q_host || !h->paper_mode) return PERCACHE_E_INVAL;
  if (cudaSetDevice(h->cfg.device) != cudaSuccess) return PERCACHE_E_CUDA;
  auto it = h->table.find(chunk_id);
  if (it == h->table.end()) return PERCACHE_E_NOTFOUND;
  const ChunkEntry& ent = it->second;
  const size_t elems = static_cast<size_t>(h->dims.n_layers) * ent.n_tokens * h->dims.q_dim;
  __nv_bfloat16* dq = nullptr;
  if (cudaMalloc(reinterpret_cast<void**>(&dq), elems * 2) != cudaSuccess) { cudaGetLastError(); return PERCACHE_E_NOMEM; }
  int rc = with_chunk_pages(h, ent.pages, [&](const int32_t* d_pages) {
    launch_chunk_pages_copy(dq, h->qpool, d_pages, ent.n_tokens, h->dims.n_layers, h->cfg.pool_pages, h->dims.q_dim, 0,
                            h->stream);
  });
  if (rc == PERCACHE_OK && cudaMemcpy(q_host, dq, elems * 2, cudaMemcpyDeviceToHost) != cudaSuccess) rc = PERCACHE_E_CUDA;
  cudaFree(dq);
  return rc;
}

int percache_prefill(percache_t* h, const percache_prompt_t* prompts, int32_t n_prompts, percache_result_t* results) {
  if (!h || !prompts || !results || n_prompts <= 0) return PERCACHE_E_INVAL;
  if (n_prompts > h->cfg.max_batch_prompts) return PERCACHE_E_CAPACITY;
  if (cudaSetDevice(h->cfg.device) != cudaSuccess) return PERCACHE_E_CUDA;
  if (!h->retained_scratch.empty()) {      // a new batch begins: the previous one can no longer be decoded on
    release_pages(h, h->retained_scratch);
    h->retained_scratch.clear();
    if (!h->plan.ctx_assembled) h->plan = Plan();
  }
  if (h->paper_mode) return prefill_paper(h, prompts, n_prompts, results);
  const auto t_host0 = std::chrono::steady_clock::now();
  const ModelDims& D = h->dims;
  const int d = D.d_model;

  // ---------------------------------------------------------------- lookup, sizes
  struct Seg { const void* src; int on_device; int row0; int n; };   // input rows to stage
  std::vector<Seg> segs;
  std::vector<std::vector<uint8_t>> hit(n_prompts);
  std::vector<int> last_hit(n_prompts, -1);                          // index of the final matched chunk, or -1
  std::unordered_map<uint64_t, std::pair<int, int>> first_miss;      // id -> (prompt, chunk) that will store it
  std::unordered_map<uint64_t, int64_t> hit_uses;                    // id -> prompt occurrences that hit it
  // Store key of every chunk: its id, or in prefix mode the key of the path of ids up to and including it.
  std::vector<std::vector<uint64_t>> keys(n_prompts);
  for (int b = 0; b < n_prompts; ++b) {
    const percache_prompt_t& P = prompts[b];
    if (P.n_chunks < 0 || (P.n_chunks > 0 && !P.chunk_ids) ||
        (P.match_mode != PERCACHE_MATCH_CHUNK_ID && P.match_mode != PERCACHE_MATCH_PREFIX_PATH))
      return PERCACHE_E_INVAL;
    keys[b].resize(static_cast<size_t>(P.n_chunks));
    uint64_t path = PATH_KEY_SEED;
    for (int i = 0; i < P.n_chunks; ++i) {
      path = path_key_step(path, P.chunk_ids[i]);
      keys[b][i] = P.match_mode == PERCACHE_MATCH_PREFIX_PATH ? path : P.chunk_ids[i];
    }
  }
  Plan plan;
  plan.cu_ctx.assign(1, 0);
  plan.cu_new.assign(1, 0);
  int64_t ctx_total = 0, new_total = 0, hit_tokens = 0, pages_needed = 0, visible_pairs = 0;
  int chunks_hit = 0, chunks_missed = 0;
  // for the gather-free form: whether every stretch of slots starts on a page boundary, how many pages the rows that
  // are not chunk content to be stored would need for the duration of the call, and the size of the page tables
  bool page_aligned = true;
  int64_t scratch_pages = 0, pt_entries = 0, max_new_per_prompt = 0;
  for (int b = 0; b < n_prompts; ++b) {
    const percache_prompt_t& P = prompts[b];
    if (P.n_query < 0 || (P.n_chunks > 0 && !P.chunk_len) || (P.n_query > 0 && !P.query_hidden))
      return PERCACHE_E_INVAL;
    hit[b].assign(static_cast<size_t>(P.n_chunks), 0);
    int64_t T = 0, n_new = 0;
    bool walking = true;      // prefix mode: the match walk stops at the first chunk that is not stored
    for (int i = 0; i < P.n_chunks; ++i) {
      const int len = P.chunk_len[i];
      if (len <= 0) return PERCACHE_E_INVAL;
      if (len % PAGE_TOKENS != 0) page_aligned = false;
      const uint64_t key = keys[b][i];
      auto it = h->table.find(key);
      const bool stored = it != h->table.end();
      if (stored && it->second.n_tokens != len) return PERCACHE_E_LEN_MISMATCH;
      if (stored && (walking || P.match_mode == PERCACHE_MATCH_CHUNK_ID)) {
        hit[b][i] = 1;
        ++chunks_hit;
        hit_tokens += len;
        ++hit_uses[key];
      } else {
        walking = false;
        if (!P.chunk_hidden || !P.chunk_hidden[i]) return PERCACHE_E_MISS_NO_INPUT;
        ++chunks_missed;
        n_new += len;
        // a node below an evicted ancestor may still be stored: it is recomputed but not stored again
        if (!stored && !first_miss.count(key)) {
          first_miss.emplace(key, std::make_pair(b, i));
          pages_needed += (len + PAGE_TOKENS - 1) / PAGE_TOKENS;
        } else {
          scratch_pages += (len + PAGE_TOKENS - 1) / PAGE_TOKENS;     // computed but not kept
        }
      }
      T += len;
    }
    // Prefix matching only: the final matched chunk gives up its last reuse_tail_drop tokens, which are computed
    // from their inputs like any new row (and not stored again: the chunk is in the store already).
    last_hit[b] = -1;
    for (int i = P.n_chunks - 1; i >= 0 && last_hit[b] < 0; --i)
      if (hit[b][i]) last_hit[b] = i;
    if (P.reuse_tail_drop != 0) {
      if (P.reuse_tail_drop < 0 || P.match_mode != PERCACHE_MATCH_PREFIX_PATH) return PERCACHE_E_INVAL;
      if (last_hit[b] >= 0) {
        if (P.reuse_tail_drop > P.chunk_len[last_hit[b]]) return PERCACHE_E_INVAL;
        if (!P.chunk_hidden || !P.chunk_hidden[last_hit[b]]) return PERCACHE_E_MISS_NO_INPUT;
        n_new += P.reuse_tail_drop;
        hit_tokens -= P.reuse_tail_drop;
        if (P.reuse_tail_drop % PAGE_TOKENS != 0) page_aligned = false;
        scratch_pages += P.reuse_tail_drop / PAGE_TOKENS;
      }
    }
    scratch_pages += (P.n_query + PAGE_TOKENS - 1) / PAGE_TOKENS;
    T += P.n_query;
    n_new += P.n_query;
    pt_entries += (T + 127) / 128 * (128 / PAGE_TOKENS);
    max_new_per_prompt = std::max(max_new_per_prompt, n_new);
    if (T <= 0) return PERCACHE_E_INVAL;
    if (T > h->cfg.max_prompt_tokens) return PERCACHE_E_CAPACITY;
    if (results[b].out_capacity_rows < n_new || (n_new > 0 && !results[b].out_hidden)) return PERCACHE_E_CAPACITY;
    ctx_total += T;
    new_total += n_new;
    if (ctx_total + static_cast<int64_t>(b + 1) * h->decode_reserve > h->ctx_cap || new_total > h->m_cap)
      return PERCACHE_E_CAPACITY;
    plan.cu_ctx.push_back(static_cast<int32_t>(ctx_total));
    plan.cu_new.push_back(static_cast<int32_t>(new_total));
  }
  // Gather-free form (paper Section 3.2.2 loads and concatenates the matched tensors; here the attention reads them
  // where they are): K and V of every slot stay in 16-token pages, the attention walks the prompt's page table and
  // rotates K on load, and the fetch -- a read, a write and a re-read of every cached K and V byte -- disappears.
  // Taken when the cached part dominates and every prompt has at most two tiles of new rows, or on request: every
  // tile of rows rotates the K blocks it reads, so the form pays off when a context block is read once or twice
  // (the fetch would move more bytes than the attention reads), not when many tiles share it.  Possible when every
  // stretch of slots is page-aligned and the tcgen05 attention runs.  The rows of the call that are not chunk
  // content to be stored then need pages of their own while the call lasts -- and beyond it when a decode reserve is
  // set: percache_decode needs the contiguous context, which its first step then assembles from the pages.
  const bool gather_free =
      page_aligned && hit_tokens > 0 && new_total > 0 &&
      !(h->flags & (PERCACHE_FLAG_REFERENCE_KERNELS | PERCACHE_FLAG_REFERENCE_ATTENTION | PERCACHE_FLAG_ALWAYS_GATHER)) &&
      static_cast<size_t>(pt_entries) <= 4 * static_cast<size_t>(h->ctx_cap) &&
      ((h->flags & PERCACHE_FLAG_GATHER_FREE) ||
       (hit_tokens >= GATHER_FREE_MIN_RATIO * new_total && max_new_per_prompt <= GATHER_FREE_MAX_NEW_ROWS));
  // with a decode reserve the decoded tokens get page slots behind every prompt's last one, so that decode steps can
  // read pages as well (an upper bound: the last page of the prompt may have room left)
  const int64_t decode_pages_per_prompt = (h->decode_reserve + PAGE_TOKENS - 1) / PAGE_TOKENS + (h->decode_reserve > 0 ? 1 : 0);
  if (gather_free) pages_needed += scratch_pages + (h->decode_reserve > 0 ? decode_pages_per_prompt * n_prompts : 0);
  // every argument check has passed: choose what would have to be evicted so that the new pages fit (never a chunk
  // this batch hits).  The store itself changes only when the device work is about to start (PageTxn::apply).
  PageTxn txn(h);
  {
    std::vector<uint64_t> victims;
    const int rc = pick_victims(h, pages_needed, hit_uses, &victims);
    if (rc < 0) return rc;
    txn.set_victims(victims);
  }
  const int evicted = static_cast<int>(txn.victims.size());
  std::vector<int32_t> scratch;                   // gather-free form: pages that only live for this call

  // ---------------------------------------------------------------- pages for the chunks that will be stored
  std::vector<std::pair<uint64_t, ChunkEntry>> pending;
  std::unordered_map<uint64_t, size_t> pending_of;
  for (int b = 0; b < n_prompts; ++b)
    for (int i = 0; i < prompts[b].n_chunks; ++i) {
      if (hit[b][i]) continue;
      const uint64_t id = keys[b][i];
      auto fm = first_miss.find(id);
      if (fm == first_miss.end() || fm->second.first != b || fm->second.second != i) continue;
      ChunkEntry ent;
      ent.n_tokens = prompts[b].chunk_len[i];
      ent.serial = h->next_serial++;
      if (txn.take((ent.n_tokens + PAGE_TOKENS - 1) / PAGE_TOKENS, &ent.pages) != PERCACHE_OK) {
        txn.undo();
        return PERCACHE_E_NOSPACE;
      }
      pending_of.emplace(id, pending.size());
      pending.emplace_back(id, std::move(ent));
    }
  // A failure before the device work leaves the store exactly as it was.  Once kernels have written pages and the
  // assembled context, the evicted chunks stay evicted, the new pages are released and the last call's context is
  // forgotten (percache_decode then refuses to continue it).
  auto fail = [&](int code) {
    if (txn.applied) h->plan = Plan();
    txn.undo();
    refresh_page_stats(h);
    return code;
  };

  // ---------------------------------------------------------------- index assembly
  const int64_t M = new_total;
  int32_t* row_slot = h->h_index;
  int32_t* row_pos = row_slot + h->m_cap;
  int32_t* row_pool = row_pos + h->m_cap;
  int32_t* row_ctx0 = row_pool + h->m_cap;
  GatherItem* items = reinterpret_cast<GatherItem*>(row_ctx0 + h->m_cap);
  AttnItem* attn_items = reinterpret_cast<AttnItem*>(reinterpret_cast<int32_t*>(items) + 4 * h->ctx_cap);
  int32_t* cta_first = reinterpret_cast<int32_t*>(attn_items) + 8 * h->max_attn_items;
  AttnMerge* merges = reinterpret_cast<AttnMerge*>(cta_first + h->n_sms + 1);
  std::vector<AttnBaseTile> base_tiles;
  int n_items = 0, n_attn_ctas = 0, n_merges = 0;
  int32_t* page_table = reinterpret_cast<int32_t*>(items);     // gather-free form: in place of the gather items
  int32_t pt_next = 0;
  std::vector<std::vector<int32_t>> decode_pages;              // per prompt: pages for tokens decoded later
  plan.slot_chunk.resize(static_cast<size_t>(ctx_total));
  plan.slot_offset.resize(static_cast<size_t>(ctx_total));
  plan.slot_is_new.resize(static_cast<size_t>(ctx_total));
  plan.row_slot.resize(static_cast<size_t>(M));
  int64_t r = 0;
  for (int b = 0; b < n_prompts; ++b) {
    const percache_prompt_t& P = prompts[b];
    const int32_t pbase = plan.cu_ctx[b];                              // index into the plan's per-slot arrays
    const int32_t ctx0 = pbase + b * h->decode_reserve;                // slot in the device context
    const int32_t pt0 = pt_next;                                       // gather-free form: first entry of its page table
    plan.ctx0.push_back(ctx0);
    plan.dec_len.push_back(0);
    int32_t t = 0;
    for (int i = 0; i <= P.n_chunks; ++i) {
      const bool is_query = (i == P.n_chunks);
      const int len = is_query ? P.n_query : P.chunk_len[i];
      if (len == 0) continue;
      const bool is_hit = !is_query && hit[b][i];
      // tokens [0, reuse_len) of the chunk come from the store, the rest (all of a missed chunk or of the query,
      // the dropped tail of the final matched chunk) are new rows
      const int reuse_len = !is_hit ? 0 : len - (i == last_hit[b] ? P.reuse_tail_drop : 0);
      for (int o = 0; o < len; ++o) {
        plan.slot_chunk[pbase + t + o] = i;
        plan.slot_offset[pbase + t + o] = o;
        plan.slot_is_new[pbase + t + o] = o < reuse_len ? 0 : 1;
      }
      if (reuse_len > 0) {
        const ChunkEntry& ent = h->table.find(keys[b][i])->second;
        if (gather_free) {
          for (int o = 0; o < reuse_len; o += PAGE_TOKENS) page_table[pt_next++] = ent.pages[o / PAGE_TOKENS];
        } else {
          for (int o = 0; o < reuse_len; o += PAGE_TOKENS) {
            GatherItem& g = items[n_items++];
            g.dst_slot = ctx0 + t + o;
            g.src_page = ent.pages[o / PAGE_TOKENS];
            g.n_tok = std::min(PAGE_TOKENS, reuse_len - o);
            g.pos = t + o;
          }
        }
      }
      if (reuse_len < len) {
        const ChunkEntry* ent = nullptr;
        if (!is_query && !is_hit) {
          auto fm = first_miss.find(keys[b][i]);
          if (fm != first_miss.end() && fm->second.first == b && fm->second.second == i)
            ent = &pending[pending_of[keys[b][i]]].second;
        }
        // gather-free form: rows that will not be stored still need page slots while the call lasts
        std::vector<int32_t> tmp_pages;
        if (gather_free && !ent) {
          if (txn.take((len - reuse_len + PAGE_TOKENS - 1) / PAGE_TOKENS, &tmp_pages) != PERCACHE_OK)
            return fail(PERCACHE_E_NOSPACE);
          scratch.insert(scratch.end(), tmp_pages.begin(), tmp_pages.end());
        }
        if (gather_free)
          for (int o = reuse_len; o < len; o += PAGE_TOKENS)
            page_table[pt_next++] = ent ? ent->pages[o / PAGE_TOKENS] : tmp_pages[(o - reuse_len) / PAGE_TOKENS];
        const char* src = static_cast<const char*>(is_query ? P.query_hidden : P.chunk_hidden[i]);
        segs.push_back(Seg{src + static_cast<size_t>(reuse_len) * d * 2, P.hidden_on_device, static_cast<int>(r),
                           len - reuse_len});
        for (int o = reuse_len; o < len; ++o, ++r) {
          row_slot[r] = ctx0 + t + o;
          row_pos[r] = t + o;
          row_pool[r] = ent ? ent->pages[o / PAGE_TOKENS] * PAGE_TOKENS + (o % PAGE_TOKENS)
                            : (gather_free ? tmp_pages[(o - reuse_len) / PAGE_TOKENS] * PAGE_TOKENS + ((o - reuse_len) % PAGE_TOKENS)
                                           : -1);
          row_ctx0[r] = ctx0;
          plan.row_slot[r] = t + o;
          visible_pairs += t + o + 1;
        }
      }
      t += len;
    }
    if (gather_free && pt_next > pt0) {     // pad the table to whole 128-slot blocks (those slots are never visible)
      const int32_t last_page = page_table[pt_next - 1];
      while ((pt_next - pt0) % (128 / PAGE_TOKENS) != 0) page_table[pt_next++] = last_page;
      if (h->decode_reserve > 0) {
        // page slots for the tokens decode steps will append: slots n_total .. n_total + reserve - 1 (the first of them
        // may still fit the prompt's last page)
        const int32_t T = plan.cu_ctx[b + 1] - plan.cu_ctx[b];
        const int32_t have = (T + PAGE_TOKENS - 1) / PAGE_TOKENS, want = (T + h->decode_reserve + PAGE_TOKENS - 1) / PAGE_TOKENS;
        std::vector<int32_t> more;
        if (want > have && txn.take(want - have, &more) != PERCACHE_OK) return fail(PERCACHE_E_NOSPACE);
        scratch.insert(scratch.end(), more.begin(), more.end());
        decode_pages.push_back(more);
      }
    }
    for (int32_t r0 = plan.cu_new[b]; r0 < plan.cu_new[b + 1]; r0 += 128) {
      AttnBaseTile a{};
      a.row0 = r0;
      a.n_rows = std::min(128, plan.cu_new[b + 1] - r0);
      a.ctx0 = gather_free ? pt0 : ctx0;           // the paged attention reads ctx0 as its page-table offset
      a.n_blocks = (row_pos[r0 + a.n_rows - 1] + 1 + 127) / 128;     // context blocks its last row can see
      base_tiles.push_back(a);
    }
  }
  {
    std::vector<AttnItem> v_items;
    std::vector<int32_t> v_first;
    std::vector<AttnMerge> v_merges;
    plan_attention(base_tiles, D.n_kv_heads * (D.n_q_heads / D.n_kv_heads / 2), h->n_sms, h->partial_slots, &v_items,
                   &v_first, &v_merges);
    if (v_items.size() > h->max_attn_items || v_merges.size() > h->max_attn_merges ||
        v_first.size() > static_cast<size_t>(h->n_sms) + 1)
      return fail(PERCACHE_E_CAPACITY);
    std::copy(v_items.begin(), v_items.end(), attn_items);
    std::fill(cta_first, cta_first + h->n_sms + 1, static_cast<int32_t>(v_items.size()));
    std::copy(v_first.begin(), v_first.end(), cta_first);
    std::copy(v_merges.begin(), v_merges.end(), merges);
    n_attn_ctas = static_cast<int>(v_first.size()) - 1;
    n_merges = static_cast<int>(v_merges.size());
  }
  const double plan_us =
      std::chrono::duration<double, std::micro>(std::chrono::steady_clock::now() - t_host0).count();

  // ---------------------------------------------------------------- device work
  // The fetch depends on nothing the layers compute (it reads pages of chunks stored by earlier
  // calls), so a large one runs beside them: one launch per layer on the side stream, and layer l's
  // attention waits for fetch l alone.  A small fetch stays one launch ahead of layer 0 (the waits
  // would cost more than they hide), and so does a phase-timed call, whose fetch time must be clean.
  const bool use_ref = (h->flags & PERCACHE_FLAG_REFERENCE_KERNELS) != 0;
  const int64_t gather_bytes = hit_tokens * D.kv_dim * 8 * D.n_layers;   // K and V, bf16 in + fp16 out
  const bool overlap_gather = n_items > 0 && M > 0 && !use_ref && !(h->flags & PERCACHE_FLAG_PHASE_TIMING) &&
                              gather_bytes >= GATHER_OVERLAP_MIN_BYTES;
  cudaStream_t s = h->stream;
  percache_stats_t& st = h->stats;
  std::memset(st.phase_us, 0, sizeof(st.phase_us));
  std::memset(st.phase_launches, 0, sizeof(st.phase_launches));
  PhaseTimer timer(h);
  bool ok = true;
  const size_t used_ints = static_cast<size_t>(reinterpret_cast<int32_t*>(merges + n_merges) - h->h_index);
  ok = ok && cudaMemcpyAsync(h->d_index, h->h_index, used_ints * sizeof(int32_t), cudaMemcpyHostToDevice, s) == cudaSuccess;
  ok = ok && cudaMemsetAsync(h->d_err, 0, sizeof(int), s) == cudaSuccess;
  const DevIndex dix = dev_index(h);
  const GatherItem* d_items = dix.items;

  if (use_ref && !h->cref) {
    const size_t wide = static_cast<size_t>(std::max(std::max(D.qkv_dim, 2 * D.d_ffn), d));
    if (!dev_alloc(h, &h->cref, static_cast<size_t>(h->m_cap) * wide)) return fail(PERCACHE_E_NOMEM);
  }
  if (h->capture_host && static_cast<int64_t>(D.n_layers + 1) * M * d > h->capture_capacity) return fail(PERCACHE_E_CAPACITY);
  txn.apply();      // from here on kernels write pages and the context

  timer.begin(PERCACHE_PH_IO);
  for (const Seg& sg : segs)
    ok = ok && cudaMemcpyAsync(h->xin + static_cast<size_t>(sg.row0) * d, sg.src, static_cast<size_t>(sg.n) * d * 2,
                               sg.on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice, s) == cudaSuccess;
  cudaEventRecord(h->ev_begin, s);
  launch_bf16_to_f32(h->xin, h->resid, M * d, s);
  timer.end();

  const size_t pool_layer = static_cast<size_t>(h->cfg.pool_pages) * PAGE_TOKENS * D.kv_dim;
  const size_t ctx_layer = static_cast<size_t>(h->ctx_cap) * D.kv_dim;
  const int Mi = static_cast<int>(M);
  if (overlap_gather) {
    ok = ok && cudaEventRecord(h->ev_fork, s) == cudaSuccess && cudaStreamWaitEvent(h->side, h->ev_fork, 0) == cudaSuccess;
    for (int l = 0; l < D.n_layers && ok; ++l) {
      launch_gather_rerope(d_items, n_items, 1, h->kpool + l * pool_layer, h->vpool + l * pool_layer, h->cfg.pool_pages,
                           h->kctx + l * ctx_layer, h->vctx + l * ctx_layer, h->ctx_cap, D.kv_dim, h->rope, h->side);
      ok = ok && cudaEventRecord(h->ev_gather[l], h->side) == cudaSuccess;
    }
  } else if (n_items > 0) {
    timer.begin(PERCACHE_PH_GATHER);
    launch_gather_rerope(d_items, n_items, D.n_layers, h->kpool, h->vpool, h->cfg.pool_pages, h->kctx, h->vctx,
                         h->ctx_cap, D.kv_dim, h->rope, s);
    timer.end();
  }
  ok = ok && (Mi <= 0 || run_layers(h, Mi, dix, n_attn_ctas, n_merges, overlap_gather, use_ref, timer, s, 0,
                                    gather_free ? reinterpret_cast<const int32_t*>(dix.items) : nullptr));
  cudaEventRecord(h->ev_end, s);
  timer.begin(PERCACHE_PH_IO);
  for (int b = 0; b < n_prompts && ok; ++b) {
    const int n_new = plan.cu_new[b + 1] - plan.cu_new[b];
    if (n_new > 0)
      ok = ok && cudaMemcpyAsync(results[b].out_hidden, h->resid + static_cast<size_t>(plan.cu_new[b]) * d,
                                 static_cast<size_t>(n_new) * d * sizeof(float),
                                 results[b].out_on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyDeviceToHost, s) == cudaSuccess;
  }
  ok = ok && cudaMemcpyAsync(h->h_err, h->d_err, sizeof(int), cudaMemcpyDeviceToHost, s) == cudaSuccess;
  timer.end();
  const cudaError_t sync_rc = cudaStreamSynchronize(s);
  if (overlap_gather && !ok) cudaStreamSynchronize(h->side);   // a failed call may have skipped the per-layer joins
  if (!ok || sync_rc != cudaSuccess || cudaGetLastError() != cudaSuccess) return fail(PERCACHE_E_CUDA);
  if (*h->h_err != 0) return fail(PERCACHE_E_DEVICE_TIMEOUT);

  // ---------------------------------------------------------------- commit
  for (auto& pe : pending) h->table.emplace(pe.first, std::move(pe.second));
  for (const auto& hu : hit_uses) h->table[hu.first].retrievals += hu.second;
  if (gather_free && h->decode_reserve > 0) {       // decode steps may follow: keep what their late assembly needs
    h->retained_scratch = scratch;
    // per prompt: the pages of its slots, then the pages for decoded tokens (the padding of the prefill table is dropped)
    int32_t at = 0;
    for (int b = 0; b < n_prompts; ++b) {
      const int32_t T = plan.cu_ctx[b + 1] - plan.cu_ctx[b];
      plan.pt0.push_back(static_cast<int32_t>(plan.page_table.size()));
      plan.page_table.insert(plan.page_table.end(), page_table + at, page_table + at + (T + PAGE_TOKENS - 1) / PAGE_TOKENS);
      plan.page_table.insert(plan.page_table.end(), decode_pages[b].begin(), decode_pages[b].end());
      at += (T + 127) / 128 * (128 / PAGE_TOKENS);
    }
  } else {
    release_pages(h, scratch);
  }
  plan.ctx_assembled = !gather_free;
  st.evictions = evicted;
  for (int b = 0; b < n_prompts; ++b) {
    results[b].n_new = plan.cu_new[b + 1] - plan.cu_new[b];
    results[b].n_total = plan.cu_ctx[b + 1] - plan.cu_ctx[b];
    if (results[b].hit_mask && prompts[b].n_chunks > 0)
      std::memcpy(results[b].hit_mask, hit[b].data(), static_cast<size_t>(prompts[b].n_chunks));
  }
  h->plan = std::move(plan);
  st.n_prompts = n_prompts;
  st.chunks_hit = chunks_hit;
  st.chunks_missed = chunks_missed;
  st.ctx_tokens = ctx_total;
  st.hit_tokens = hit_tokens;
  st.new_rows = new_total;
  refresh_page_stats(h);
  st.host_plan_us = plan_us;
  st.attn_visible_pairs = visible_pairs;
  st.gather_free = gather_free ? 1 : 0;
  float ms = 0.f;
  cudaEventElapsedTime(&ms, h->ev_begin, h->ev_end);
  st.device_us = 1000.0 * ms;
  timer.collect();
  return PERCACHE_OK;
}

int percache_debug_capture_layers(percache_t* h, float* host_buf, int64_t capacity_floats) {
  if (!h || (host_buf && capacity_floats <= 0)) return PERCACHE_E_INVAL;
  h->capture_host = host_buf;
  h->capture_capacity = host_buf ? capacity_floats : 0;
  return PERCACHE_OK;
}

int percache_set_decode_reserve(percache_t* h, int32_t tokens_per_prompt) {
  if (!h || tokens_per_prompt < 0) return PERCACHE_E_INVAL;
  h->decode_reserve = tokens_per_prompt;
  return PERCACHE_OK;
}

int percache_decode(percache_t* h, int32_t n_prompts, const void* hidden, int32_t hidden_on_device, float* out_hidden,
                    int32_t out_on_device) {
  if (!h || !hidden || !out_hidden || n_prompts <= 0 || h->paper_mode) return PERCACHE_E_INVAL;
  Plan& plan = h->plan;
  if (static_cast<size_t>(n_prompts) + 1 != plan.cu_ctx.size()) return PERCACHE_E_INVAL;   // not the last call's batch
  // the last prefill ran gather-free: without a decode reserve nothing was kept to build the context from
  if (!plan.ctx_assembled && plan.page_table.empty()) return PERCACHE_E_INVAL;
  if (n_prompts > h->m_cap) return PERCACHE_E_CAPACITY;
  if (cudaSetDevice(h->cfg.device) != cudaSuccess) return PERCACHE_E_CUDA;
  const auto t_host0 = std::chrono::steady_clock::now();
  const ModelDims& D = h->dims;
  const int d = D.d_model;
  int32_t* row_slot = h->h_index;
  int32_t* row_pos = row_slot + h->m_cap;
  int32_t* row_pool = row_pos + h->m_cap;
  int32_t* row_ctx0 = row_pool + h->m_cap;
  GatherItem* items = reinterpret_cast<GatherItem*>(row_ctx0 + h->m_cap);
  AttnItem* attn_items = reinterpret_cast<AttnItem*>(reinterpret_cast<int32_t*>(items) + 4 * h->ctx_cap);
  int32_t* cta_first = reinterpret_cast<int32_t*>(attn_items) + 8 * h->max_attn_items;
  AttnMerge* merges = reinterpret_cast<AttnMerge*>(cta_first + h->n_sms + 1);
  std::vector<AttnBaseTile> base_tiles;
  int64_t visible_pairs = 0;
  for (int b = 0; b < n_prompts; ++b) {
    const int32_t T = plan.cu_ctx[b + 1] - plan.cu_ctx[b] + plan.dec_len[b];     // tokens so far = the new position
    if (plan.dec_len[b] >= h->decode_reserve || T + 1 > h->cfg.max_prompt_tokens) return PERCACHE_E_CAPACITY;
    row_slot[b] = plan.ctx0[b] + T;
    row_pos[b] = T;
    row_pool[b] = -1;                       // decoded tokens are not chunk content: nothing goes to the store
    if (!plan.ctx_assembled)                // ... but after a gather-free prefill they get a page slot lent to the batch
      row_pool[b] = plan.page_table[static_cast<size_t>(plan.pt0[b] + T / PAGE_TOKENS)] * PAGE_TOKENS + T % PAGE_TOKENS;
    row_ctx0[b] = plan.ctx0[b];
    base_tiles.push_back(AttnBaseTile{b, 1, plan.ctx0[b], (T + 1 + 127) / 128});
    visible_pairs += T + 1;
  }
  // One query row per prompt: the attention is a matter of reading every prompt's K and V once, which the
  // weight-streaming style kernel of attn_decode.cu does on the CUDA cores; (prompt, KV head) pairs are cut into
  // chunks of context slots so that a few hundred blocks per SM-full are in flight.
  const int group = D.n_q_heads / D.n_kv_heads;
  const bool stream_attention = !(h->flags & (PERCACHE_FLAG_REFERENCE_KERNELS | PERCACHE_FLAG_REFERENCE_ATTENTION |
                                              PERCACHE_FLAG_NO_SMALL_ROW_KERNELS)) && (group == 2 || group == 4);
  // After a gather-free prefill the first decode step assembles the context (the fetch the prefill skipped, over every
  // slot) and decoding goes on as usual.  With PERCACHE_FLAG_GATHER_FREE set, the streaming kernel reads the pages
  // themselves instead (K rotated on load) and no context is ever assembled for this batch: every step's attention is
  // then about 40 % slower (measured), so this pays only for a handful of decoded tokens.
  const bool paged_decode = !plan.ctx_assembled && stream_attention && (h->flags & PERCACHE_FLAG_GATHER_FREE);
  int n_attn_ctas = 0, n_merges = 0, n_decode_items = 0;
  if (stream_attention) {
    int64_t total_slots = 0;
    for (int b = 0; b < n_prompts; ++b) total_slots += row_pos[b] + 1;
    int chunk = static_cast<int>(std::min<int64_t>(1024, std::max<int64_t>(64, (total_slots * D.n_kv_heads / (4 * h->n_sms) + 63) / 64 * 64)));
    const size_t scratch_items = static_cast<size_t>(h->partial_slots) * 2 * 128 * HEAD_DIM / (static_cast<size_t>(group) * HEAD_DIM);
    auto count_items = [&](int ch) {
      int64_t n = 0;
      for (int b = 0; b < n_prompts; ++b) n += static_cast<int64_t>((row_pos[b] + 1 + ch - 1) / ch) * D.n_kv_heads;
      return n;
    };
    while (static_cast<size_t>(count_items(chunk)) > std::min(h->max_attn_items, scratch_items)) chunk *= 2;
    if (static_cast<size_t>(n_prompts) * D.n_kv_heads > h->max_attn_merges) return PERCACHE_E_CAPACITY;
    DecodeAttnItem* ditems = reinterpret_cast<DecodeAttnItem*>(attn_items);
    DecodeAttnMerge* dmerges = reinterpret_cast<DecodeAttnMerge*>(merges);
    // Items are ordered (prompt, chunk, KV head): the blocks of the KV heads of one chunk run side by side and
    // together read whole 2 KB context rows, which keeps DRAM pages open; the results of a (prompt, KV head) still
    // go to consecutive slots for the merge.
    int next_slot = 0;
    for (int b = 0; b < n_prompts; ++b) {
      const int n_slots = row_pos[b] + 1;
      const int n_chunks = (n_slots + chunk - 1) / chunk;
      for (int g = 0; g < D.n_kv_heads; ++g)
        dmerges[n_merges++] = DecodeAttnMerge{b, g, next_slot + g * n_chunks, n_chunks, 0, 0, 0, 0};
      for (int c = 0; c < n_chunks; ++c)
        for (int g = 0; g < D.n_kv_heads; ++g)
          ditems[n_decode_items++] = DecodeAttnItem{b, paged_decode ? plan.pt0[b] : plan.ctx0[b], c * chunk,
                                                    std::min(n_slots, (c + 1) * chunk), g, next_slot + g * n_chunks + c, 0, 0};
      next_slot += n_chunks * D.n_kv_heads;
    }
  } else {
    std::vector<AttnItem> v_items;
    std::vector<int32_t> v_first;
    std::vector<AttnMerge> v_merges;
    plan_attention(base_tiles, D.n_kv_heads * (D.n_q_heads / D.n_kv_heads / 2), h->n_sms, h->partial_slots, &v_items,
                   &v_first, &v_merges);
    if (v_items.size() > h->max_attn_items || v_merges.size() > h->max_attn_merges ||
        v_first.size() > static_cast<size_t>(h->n_sms) + 1)
      return PERCACHE_E_CAPACITY;
    std::copy(v_items.begin(), v_items.end(), attn_items);
    std::fill(cta_first, cta_first + h->n_sms + 1, static_cast<int32_t>(v_items.size()));
    std::copy(v_first.begin(), v_first.end(), cta_first);
    std::copy(v_merges.begin(), v_merges.end(), merges);
    n_attn_ctas = static_cast<int>(v_first.size()) - 1;
    n_merges = static_cast<int>(v_merges.size());
  }
  const double plan_us =
      std::chrono::duration<double, std::micro>(std::chrono::steady_clock::now() - t_host0).count();

  cudaStream_t s = h->stream;
  percache_stats_t& st = h->stats;
  std::memset(st.phase_us, 0, sizeof(st.phase_us));
  std::memset(st.phase_launches, 0, sizeof(st.phase_launches));
  PhaseTimer timer(h);
  const bool use_ref = (h->flags & PERCACHE_FLAG_REFERENCE_KERNELS) != 0;
  if (use_ref && !h->cref) {
    const size_t wide = static_cast<size_t>(std::max(std::max(D.qkv_dim, 2 * D.d_ffn), d));
    if (!dev_alloc(h, &h->cref, static_cast<size_t>(h->m_cap) * wide)) return PERCACHE_E_NOMEM;
  }
  bool ok = true;
  bool assembled_now = false;
  if (paged_decode) {       // the prompts' page tables (with the decoded tokens' pages) in place of the gather items
    if (plan.page_table.size() > 4 * static_cast<size_t>(h->ctx_cap)) return PERCACHE_E_CAPACITY;
    std::memcpy(items, plan.page_table.data(), plan.page_table.size() * sizeof(int32_t));
  } else if (!plan.ctx_assembled) {
    // First decode step after a gather-free prefill: every slot of every prompt still sits in a page (cached chunks
    // in theirs, the rows that prefill computed in the pages lent to them), so the fetch that prefill skipped runs
    // now, over all slots, and builds the contiguous context the decode kernels read and append to.
    int n_items = 0;
    for (int b = 0; b < n_prompts; ++b) {
      const int32_t T = plan.cu_ctx[b + 1] - plan.cu_ctx[b];
      for (int32_t o = 0; o < T; o += PAGE_TOKENS) {
        GatherItem& g = items[n_items++];
        g.dst_slot = plan.ctx0[b] + o;
        g.src_page = plan.page_table[static_cast<size_t>(plan.pt0[b] + o / PAGE_TOKENS)];
        g.n_tok = std::min<int32_t>(PAGE_TOKENS, T - o);
        g.pos = o;
      }
    }
    ok = ok && cudaMemcpyAsync(reinterpret_cast<int32_t*>(const_cast<GatherItem*>(dev_index(h).items)), items,
                               static_cast<size_t>(n_items) * sizeof(GatherItem), cudaMemcpyHostToDevice, s) == cudaSuccess;
    timer.begin(PERCACHE_PH_GATHER);
    launch_gather_rerope(dev_index(h).items, n_items, D.n_layers, h->kpool, h->vpool, h->cfg.pool_pages, h->kctx, h->vctx,
                         h->ctx_cap, D.kv_dim, h->rope, s);
    timer.end();
    assembled_now = true;
  }
  const size_t used_ints = static_cast<size_t>(reinterpret_cast<int32_t*>(merges + n_merges) - h->h_index);
  ok = ok && cudaMemcpyAsync(h->d_index, h->h_index, used_ints * sizeof(int32_t), cudaMemcpyHostToDevice, s) == cudaSuccess;
  ok = ok && cudaMemsetAsync(h->d_err, 0, sizeof(int), s) == cudaSuccess;
  timer.begin(PERCACHE_PH_IO);
  ok = ok && cudaMemcpyAsync(h->xin, hidden, static_cast<size_t>(n_prompts) * d * 2,
                             hidden_on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice, s) == cudaSuccess;
  cudaEventRecord(h->ev_begin, s);
  launch_bf16_to_f32(h->xin, h->resid, static_cast<int64_t>(n_prompts) * d, s);
  timer.end();
  ok = ok && run_layers(h, n_prompts, dev_index(h), n_attn_ctas, n_merges, false, use_ref, timer, s, n_decode_items,
                        paged_decode ? reinterpret_cast<const int32_t*>(dev_index(h).items) : nullptr);
  cudaEventRecord(h->ev_end, s);
  timer.begin(PERCACHE_PH_IO);
  ok = ok && cudaMemcpyAsync(out_hidden, h->resid, static_cast<size_t>(n_prompts) * d * sizeof(float),
                             out_on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyDeviceToHost, s) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(h->h_err, h->d_err, sizeof(int), cudaMemcpyDeviceToHost, s) == cudaSuccess;
  timer.end();
  const cudaError_t sync_rc = cudaStreamSynchronize(s);
  if (!ok || sync_rc != cudaSuccess || cudaGetLastError() != cudaSuccess) return PERCACHE_E_CUDA;
  if (*h->h_err != 0) return PERCACHE_E_DEVICE_TIMEOUT;
  if (assembled_now) {         // the context exists now: the lent pages go back
    plan.ctx_assembled = true;
    plan.page_table.clear();
    plan.pt0.clear();
    release_pages(h, h->retained_scratch);
    h->retained_scratch.clear();
    refresh_page_stats(h);
  }
  for (int b = 0; b < n_prompts; ++b) plan.dec_len[b] += 1;      // the token's K/V now is part of the context
  st.n_prompts = n_prompts;
  st.chunks_hit = st.chunks_missed = 0;
  st.hit_tokens = 0;
  st.new_rows = n_prompts;
  st.ctx_tokens = 0;
  for (int b = 0; b < n_prompts; ++b) st.ctx_tokens += plan.cu_ctx[b + 1] - plan.cu_ctx[b] + plan.dec_len[b];
  st.host_plan_us = plan_us;
  st.attn_visible_pairs = visible_pairs;
  st.evictions = 0;
  st.gather_free = 0;
  float ms = 0.f;
  cudaEventElapsedTime(&ms, h->ev_begin, h->ev_end);
  st.device_us = 1000.0 * ms;
  timer.collect();
  return PERCACHE_OK;
}

int percache_get_stats(percache_t* h, percache_stats_t* out) {
  if (!h || !out) return PERCACHE_E_INVAL;
  *out = h->stats;
  return PERCACHE_OK;
}

int percache_debug_attn_plan(const int32_t* n_blocks, int32_t n_tiles, int32_t units_per_tile, int32_t n_ctas,
                             int32_t max_partial_slots, int32_t* items_out, int64_t items_capacity,
                             int64_t* counts_out) {
  if (n_tiles < 0 || units_per_tile <= 0 || n_ctas <= 0 || max_partial_slots < 0 || !counts_out ||
      (n_tiles > 0 && !n_blocks))
    return PERCACHE_E_INVAL;
  std::vector<AttnBaseTile> tiles(static_cast<size_t>(n_tiles));
  for (int i = 0; i < n_tiles; ++i) {
    if (n_blocks[i] <= 0) return PERCACHE_E_INVAL;
    tiles[static_cast<size_t>(i)] = AttnBaseTile{i * 128, 128, 0, n_blocks[i]};   // row0 identifies the tile
  }
  std::vector<AttnItem> items;
  std::vector<int32_t> first;
  std::vector<AttnMerge> merges;
  const int64_t makespan = plan_attention(tiles, units_per_tile, n_ctas, max_partial_slots, &items, &first, &merges);
  counts_out[0] = static_cast<int64_t>(items.size());
  counts_out[1] = static_cast<int64_t>(first.size()) - 1;
  counts_out[2] = static_cast<int64_t>(merges.size());
  counts_out[3] = makespan;
  if (static_cast<int64_t>(items.size()) > items_capacity || (!items.empty() && !items_out)) return PERCACHE_E_CAPACITY;
  size_t cta = 0;
  for (size_t i = 0; i < items.size(); ++i) {
    while (cta + 1 < first.size() && static_cast<int32_t>(i) >= first[cta + 1]) ++cta;
    int32_t* o = items_out + 6 * i;
    o[0] = items[i].row0 / 128; o[1] = items[i].unit; o[2] = items[i].blk_begin; o[3] = items[i].blk_end;
    o[4] = items[i].partial_slot; o[5] = static_cast<int32_t>(cta);
  }
  return PERCACHE_OK;
}

int64_t percache_debug_read_plan(percache_t* h, int32_t which, int32_t* out, int64_t capacity) {
  if (!h || !out) return PERCACHE_E_INVAL;
  const std::vector<int32_t>* v = nullptr;
  switch (which) {
    case 0: v = &h->plan.cu_ctx; break;
    case 1: v = &h->plan.cu_new; break;
    case 2: v = &h->plan.slot_chunk; break;
    case 3: v = &h->plan.slot_offset; break;
    case 4: v = &h->plan.slot_is_new; break;
    case 5: v = &h->plan.row_slot; break;
    default: return PERCACHE_E_INVAL;
  }
  if (static_cast<int64_t>(v->size()) > capacity) return PERCACHE_E_CAPACITY;
  if (!v->empty()) std::memcpy(out, v->data(), v->size() * sizeof(int32_t));
  return static_cast<int64_t>(v->size());
}

int percache_debug_read_ctx(percache_t* h, int32_t prompt, int32_t layer, void* k_host, void* v_host,
                            int64_t capacity_tokens) {
  if (!h || !k_host || !v_host || layer < 0 || layer >= h->dims.n_layers || prompt < 0 ||
      prompt + 1 >= static_cast<int32_t>(h->plan.cu_ctx.size()) || !h->plan.ctx_assembled || h->paper_mode)
    return PERCACHE_E_INVAL;
  if (cudaSetDevice(h->cfg.device) != cudaSuccess) return PERCACHE_E_CUDA;
  const size_t ctx_layer = static_cast<size_t>(h->ctx_cap) * h->dims.kv_dim;
  const size_t off = layer * ctx_layer + static_cast<size_t>(h->plan.ctx0[prompt]) * h->dims.kv_dim;
  const int64_t tokens = h->plan.cu_ctx[prompt + 1] - h->plan.cu_ctx[prompt] + h->plan.dec_len[prompt];
  if (capacity_tokens < tokens) return PERCACHE_E_CAPACITY;
  const size_t bytes = static_cast<size_t>(tokens) * h->dims.kv_dim * 2;
  if (cudaMemcpy(k_host, h->kctx + off, bytes, cudaMemcpyDeviceToHost) != cudaSuccess ||
      cudaMemcpy(v_host, h->vctx + off, bytes, cudaMemcpyDeviceToHost) != cudaSuccess)
    return PERCACHE_E_CUDA;
  return PERCACHE_OK;
}

int percache_debug_gemm(int32_t device, int32_t M, int32_t N, int32_t K, const void* a_f16, const void* b_f16,
                        float* c, int32_t use_reference) {
  if (M <= 0 || N <= 0 || K <= 0 || !a_f16 || !b_f16 || !c) return PERCACHE_E_INVAL;
  if (use_reference < 0 || use_reference > 2) return PERCACHE_E_INVAL;
  if (use_reference != 1 && (K % 64 != 0 || N % 128 != 0)) return PERCACHE_E_INVAL;
  if (use_reference == 2 && N % 256 != 0) return PERCACHE_E_INVAL;
  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || device < 0 || device >= n_dev) { cudaGetLastError(); return PERCACHE_E_CUDA; }
  if (cudaSetDevice(device) != cudaSuccess) { cudaGetLastError(); return PERCACHE_E_CUDA; }
  if (init_driver_api() != 0) return PERCACHE_E_CUDA;
  __half *dA = nullptr, *dB = nullptr;
  float* dC = nullptr;
  int *dErr = nullptr, hErr = 0;
  int rc = PERCACHE_OK;
  const size_t m_pad = static_cast<size_t>((M + 255) / 256) * 256;
  if (cudaMalloc(reinterpret_cast<void**>(&dA), m_pad * K * 2) != cudaSuccess ||
      cudaMalloc(reinterpret_cast<void**>(&dB), static_cast<size_t>(N) * K * 2) != cudaSuccess ||
      cudaMalloc(reinterpret_cast<void**>(&dC), static_cast<size_t>(M) * N * 4) != cudaSuccess ||
      cudaMalloc(reinterpret_cast<void**>(&dErr), sizeof(int)) != cudaSuccess) {
    cudaGetLastError();
    rc = PERCACHE_E_NOMEM;
  }
  if (rc == PERCACHE_OK) {
    cudaMemset(dA, 0, m_pad * K * 2);
    cudaMemset(dErr, 0, sizeof(int));
    cudaMemcpy(dA, a_f16, static_cast<size_t>(M) * K * 2, cudaMemcpyHostToDevice);
    cudaMemcpy(dB, b_f16, static_cast<size_t>(N) * K * 2, cudaMemcpyHostToDevice);
    if (use_reference == 1) {
      launch_ref_gemm(dA, dB, dC, M, N, K, nullptr);
    } else {
      GemmOperand mA, mB;
      int n_sms = 148;
      cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, device);
      const int pair = use_reference == 2 ? 1 : 0;
      const int bn = pair || (N % 256 == 0 && M >= 512) ? 256 : 128;     // both tile widths get exercised by the tests
      if (make_operand_map(&mA, dA, static_cast<int64_t>(m_pad), K, 128) != 0 ||
          make_operand_map(&mB, dB, N, K, pair ? 128 : bn) != 0 ||
          launch_umma_gemm(mA, mB, M, N, K, bn, EPI_STORE_F32, nullptr, dC, dErr, n_sms, nullptr, 1, pair) != 0)
        rc = PERCACHE_E_CUDA;
    }
    if (rc == PERCACHE_OK && (cudaDeviceSynchronize() != cudaSuccess || cudaGetLastError() != cudaSuccess)) rc = PERCACHE_E_CUDA;
    if (rc == PERCACHE_OK) {
      cudaMemcpy(&hErr, dErr, sizeof(int), cudaMemcpyDeviceToHost);
      if (hErr != 0) rc = PERCACHE_E_DEVICE_TIMEOUT;
      else if (cudaMemcpy(c, dC, static_cast<size_t>(M) * N * 4, cudaMemcpyDeviceToHost) != cudaSuccess) rc = PERCACHE_E_CUDA;
    }
  }
  if (dA) cudaFree(dA);
  if (dB) cudaFree(dB);
  if (dC) cudaFree(dC);
  if (dErr) cudaFree(dErr);
  return rc;
}

}  // extern "C"
