// Host side of libhb: context, workspace carve-up, page / slot free lists, descriptor
// validation and packing, and the launch sequence of one mixed step (the Forward, IncPooler
// and logits part of the paper's inference loop, Algorithm 1).
#include <math.h>
#include <string.h>

#include <algorithm>
#include <new>

#include "hb_internal.h"

namespace {

constexpr int POOL_ROWS = 32;   // rows per pooling work item
constexpr int ATT_TILE_ROWS = 64;   // sizing only: the item list is reserved for chunk tiles as short as this
constexpr int ATT_TC_ROWS = 128;    // query rows per tcgen05 chunk attention item
// Keys per decode attention item (a row's keys are cut into about this many per split; the count depends
// on the row's own context and this value only).  A split costs a partial record, a fence, an atomic and
// a share of the merge: with the attention blocks resident and the chunk tiles filling the tail of the
// launch, 2048 measured 6 % faster than 1024 on the decode items of the 7B mixed step and 8-12 % faster
// per step on the sweep's mixes (contexts of 2048: no split at all); 1024 keeps more blocks busy when a
// step holds only a few long decode rows.  Process-wide, read when a context is created.
int g_att_split_keys = 2048;
constexpr int N_STAGING = 4;    // pinned descriptor staging ring

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

bool misaligned(const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) != 0; }

bool cfg_ok(const hb_model_cfg* c) {
  if (!c) return false;
  if (c->n_layers < 1 || c->d_model < 64 || c->n_heads < 1 || c->n_kv_heads < 1 || c->d_ffn < 64 || c->vocab < 8)
    return false;
  if (c->head_dim != 64 && c->head_dim != 128) return false;
  if (c->n_heads % c->n_kv_heads) return false;
  const int g = c->n_heads / c->n_kv_heads;
  if (g > 16 || (64 % g)) return false;  // attention tiles: 64 rows = (64/g) tokens x g heads
  if (c->d_model % 64 || (c->n_heads * c->head_dim) % 64 || c->d_ffn % 64 || c->vocab % 8) return false;
  if (c->d_model > 8192) return false;
  if (c->page_size != 16) return false;
  if (c->max_pos < 1 || !(c->rope_theta > 0.f) || !(c->rms_eps >= 0.f)) return false;
  return true;
}

struct Carve {
  size_t off = 0;
  size_t take(size_t bytes) {
    const size_t o = off;
    off = align_up(off + bytes, 256);
    return o;
  }
};

struct Layout {
  size_t x, h, q, attn_out, act, lora_u, lora_part, lora_counters, resid_turns, logit_in, rope_cos, rope_sin, attn_part, pool_part, counters, attn_counters,
      status, desc;
  size_t total, desc_cap, attn_part_floats, pool_part_floats;
  int32_t rows_pad, logit_rows_pad, n_counters, max_pool_items, max_attn_items, n_resid_turns;
  int32_t split_keys;   // keys per decode attention item of this context
};

Layout make_layout(const hb_model_cfg& c, int32_t max_tokens, int32_t max_segs, int32_t max_page_ids) {
  Layout L{};
  Carve cv;
  const size_t rows = align_up(static_cast<size_t>(max_tokens), 128);
  const size_t lrows = align_up(static_cast<size_t>(max_segs), 128);
  const size_t n_q = static_cast<size_t>(c.n_heads) * c.head_dim;
  L.rows_pad = static_cast<int32_t>(rows);
  L.logit_rows_pad = static_cast<int32_t>(lrows);
  L.x = cv.take(rows * c.d_model * 4);
  L.h = cv.take(rows * c.d_model * 2);
  L.q = cv.take(rows * n_q * 2);
  L.attn_out = cv.take(rows * n_q * 2);
  L.act = cv.take(rows * c.d_ffn * 2);
  L.lora_u = cv.take(rows * HB_LORA_U_COLS * 2);
  L.lora_part = cv.take(static_cast<size_t>(HB_LORA_K_SPLITS) * rows * HB_LORA_U_COLS * 4);
  L.lora_counters = cv.take((rows / 128) * 2 * 8 * 4);
  // one word per (128-row block, column tile, epilogue warp); the narrowest column tile is 128 wide
  L.n_resid_turns = static_cast<int32_t>((rows / 128) * ((static_cast<size_t>(c.d_model) + 127) / 128) * 8);
  L.resid_turns = cv.take(static_cast<size_t>(L.n_resid_turns) * 4);
  L.logit_in = cv.take(lrows * 2 * c.d_model * 2);
  L.rope_cos = cv.take(static_cast<size_t>(c.max_pos) * (c.head_dim / 2) * 4);
  L.rope_sin = cv.take(static_cast<size_t>(c.max_pos) * (c.head_dim / 2) * 4);
  L.max_pool_items = max_tokens / POOL_ROWS + max_segs + 1;
  const int G = c.n_heads / c.n_kv_heads;
  L.split_keys = g_att_split_keys;
  const int max_splits = (c.max_pos + L.split_keys - 1) / L.split_keys;
  L.max_attn_items = c.n_kv_heads * (max_tokens * G / ATT_TILE_ROWS + max_segs + max_segs * max_splits);
  L.attn_part_floats = static_cast<size_t>(max_segs) * c.n_kv_heads * max_splits * G * (c.head_dim + 2);
  L.pool_part_floats = static_cast<size_t>(L.max_pool_items) * c.d_model;
  L.attn_part = cv.take(L.attn_part_floats * 4);
  L.pool_part = cv.take(L.pool_part_floats * 4);
  L.n_counters = max_segs + 1;
  L.counters = cv.take(static_cast<size_t>(L.n_counters) * 4);
  L.attn_counters = cv.take(static_cast<size_t>(max_segs) * c.n_kv_heads * 4);
  L.status = cv.take(256);
  size_t dc = 0;
  dc += align_up(static_cast<size_t>(max_tokens) * 4, 16) * 4;          // tok, row_seg, row_pos, row_page
  dc += align_up(static_cast<size_t>(max_segs) * sizeof(hb_seg), 16);
  dc += align_up(static_cast<size_t>(max_page_ids) * 4, 16);
  dc += align_up(static_cast<size_t>(max_segs) * 4, 16);                // logit_src
  dc += align_up(static_cast<size_t>(L.max_attn_items) * sizeof(AttnItem), 16);
  dc += align_up(static_cast<size_t>(L.max_pool_items) * sizeof(PoolItem), 16);
  L.desc_cap = dc + 128;
  L.desc = cv.take(L.desc_cap);
  L.total = cv.off;
  return L;
}

// Marks the validation needs (one byte per page / slot / output row).  A context keeps one and
// reuses it, so that a step allocates host memory only when it meets a larger cache than any before.
struct ValidateScratch {
  std::vector<uint8_t> page_written, slot_used, lrow, erow;
  static void zeroed(std::vector<uint8_t>& v, size_t n) {
    if (v.size() < n) v.resize(n);
    memset(v.data(), 0, n);
  }
};

int validate(const hb_model_cfg& c, int32_t max_tokens, int32_t max_segs, int32_t max_page_ids, int32_t n_pages,
             int32_t n_slots, int32_t rowbuf_rows, const hb_batch_desc* d, ValidateScratch& vs) {
  if (!d) return HB_ERR_BAD_ARG;
  if (d->n_tokens < 0 || d->n_segs < 0 || d->n_page_ids < 0 || d->n_logit_rows < 0 || d->n_emb_rows < 0)
    return HB_ERR_BAD_DESC;
  if (d->n_tokens > max_tokens || d->n_segs > max_segs || d->n_page_ids > max_page_ids) return HB_ERR_TOO_LARGE;
  if ((d->n_tokens > 0 && !d->token_ids) || (d->n_segs > 0 && !d->segs) || (d->n_page_ids > 0 && !d->page_ids))
    return HB_ERR_BAD_ARG;
  if ((d->n_tokens == 0) != (d->n_segs == 0)) return HB_ERR_BAD_DESC;
  for (int32_t t = 0; t < d->n_tokens; ++t)
    if (d->token_ids[t] < 0 || d->token_ids[t] >= c.vocab) return HB_ERR_BAD_DESC;
  for (int32_t i = 0; i < d->n_page_ids; ++i)
    if (d->page_ids[i] < 0 || d->page_ids[i] >= n_pages) return HB_ERR_BAD_DESC;
  const int P = c.page_size;
  ValidateScratch::zeroed(vs.page_written, static_cast<size_t>(std::max(n_pages, 1)));
  ValidateScratch::zeroed(vs.slot_used, static_cast<size_t>(std::max(n_slots, 1)));
  ValidateScratch::zeroed(vs.lrow, static_cast<size_t>(std::max(d->n_logit_rows, 1)));
  ValidateScratch::zeroed(vs.erow, static_cast<size_t>(std::max(d->n_emb_rows, 1)));
  uint8_t* page_written = vs.page_written.data();
  uint8_t* slot_used = vs.slot_used.data();
  uint8_t* lrow = vs.lrow.data();
  uint8_t* erow = vs.erow.data();
  int32_t at = 0, prev_kind = 0, n_l = 0, n_e = 0;
  for (int32_t r = 0; r < d->n_segs; ++r) {
    const hb_seg& s = d->segs[r];
    if (s.kind < HB_KIND_DECODE || s.kind > HB_KIND_EMBED_CHUNK || s.kind < prev_kind) return HB_ERR_BAD_DESC;
    prev_kind = s.kind;
    if (s.q_start != at || s.q_len < 1 || (s.kind == HB_KIND_DECODE && s.q_len != 1)) return HB_ERR_BAD_DESC;
    if (s.q_len > d->n_tokens - at) return HB_ERR_BAD_DESC;
    at += s.q_len;
    if (s.pos_start < 0 || s.pos_start > c.max_pos - s.q_len) return HB_ERR_BAD_DESC;
    const int32_t need = (s.pos_start + s.q_len + P - 1) / P;
    if (s.pt_start < 0 || s.pt_len < need || s.pt_start > d->n_page_ids - s.pt_len) return HB_ERR_BAD_DESC;
    // pages this segment writes must not be listed by any other segment, nor twice by this one
    for (int32_t b = s.pos_start / P; b < need; ++b) {
      const int32_t pg = d->page_ids[s.pt_start + b];
      if (page_written[pg]) return HB_ERR_BAD_DESC;
      page_written[pg] = static_cast<uint8_t>(1);
    }
    const bool embed = (s.kind == HB_KIND_EMBED_CHUNK);
    if (embed) {
      if (s.pool_mode < HB_POOL_MEAN || s.pool_mode > HB_POOL_MAX) return HB_ERR_BAD_DESC;
      // a buffered head keeps every row of the request: the whole text must fit the slot's row buffer
      if (s.pool_mode == HB_POOL_MAX && s.pos_start + s.q_len > rowbuf_rows) return HB_ERR_BAD_DESC;
      if (s.pool_slot < 0 || s.pool_slot >= n_slots || slot_used[s.pool_slot]) return HB_ERR_BAD_DESC;
      slot_used[s.pool_slot] = 1;
      if (s.logits_row != -1) return HB_ERR_BAD_DESC;
      if (s.is_final) {
        if (s.emb_row < 0 || s.emb_row >= d->n_emb_rows || erow[s.emb_row]) return HB_ERR_BAD_DESC;
        erow[s.emb_row] = 1;
        ++n_e;
      } else if (s.emb_row != -1) {
        return HB_ERR_BAD_DESC;
      }
    } else {
      if (s.pool_mode != HB_POOL_NONE || s.pool_slot != -1 || s.emb_row != -1) return HB_ERR_BAD_DESC;
      const bool wants = (s.kind == HB_KIND_DECODE) || (s.is_final != 0);
      if (wants) {
        if (s.logits_row < 0 || s.logits_row >= d->n_logit_rows || lrow[s.logits_row]) return HB_ERR_BAD_DESC;
        lrow[s.logits_row] = 1;
        ++n_l;
      } else if (s.logits_row != -1) {
        return HB_ERR_BAD_DESC;
      }
    }
  }
  if (at != d->n_tokens || n_l != d->n_logit_rows || n_e != d->n_emb_rows) return HB_ERR_BAD_DESC;
  // a page read by one segment and written by another: reject (read-only sharing is allowed)
  for (int32_t r = 0; r < d->n_segs; ++r) {
    const hb_seg& s = d->segs[r];
    const int32_t first_w = s.pos_start / P;
    for (int32_t b = 0; b < first_w && b < s.pt_len; ++b)
      if (page_written[d->page_ids[s.pt_start + b]]) return HB_ERR_BAD_DESC;
  }
  return HB_OK;
}

struct Staging {
  uint8_t* host = nullptr;
  cudaEvent_t ev = nullptr;
  bool pending = false;
};

struct ProfRec {
  cudaEvent_t a, b;
  int cls;
};

struct CtxExtra {
  Staging ring[N_STAGING];
  int next = 0;
  Layout lay;
  bool profiling = false;
  std::vector<ProfRec> free_recs, used_recs;
  // host scratch of a step, reserved at hb_create for the context's limits and reused by every call
  ValidateScratch vscratch;
  std::vector<PoolItem> pitems;
  std::vector<AttnItem> aitems, titems;
  std::vector<uint64_t> sort_keys;
};

CtxExtra* extra_of(hb_ctx* c) { return static_cast<CtxExtra*>(c->extra); }

}  // namespace

extern "C" {

int hb_workspace_bytes(const hb_model_cfg* cfg, int32_t max_tokens, int32_t max_segs, int32_t max_page_ids,
                       size_t* out_bytes) {
  if (!cfg_ok(cfg) || !out_bytes || max_tokens < 1 || max_segs < 1 || max_page_ids < 1) return HB_ERR_BAD_ARG;
  *out_bytes = make_layout(*cfg, max_tokens, max_segs, max_page_ids).total;
  return HB_OK;
}

int hb_create(const hb_model_cfg* cfg, int32_t max_tokens, int32_t max_segs, int32_t max_page_ids, void* workspace,
              size_t workspace_bytes, hb_ctx** out) {
  if (!out) return HB_ERR_BAD_ARG;
  *out = nullptr;
  if (!cfg) return HB_ERR_BAD_ARG;
  if (!cfg_ok(cfg)) return HB_ERR_UNSUPPORTED;
  if (max_tokens < 1 || max_segs < 1 || max_page_ids < 1) return HB_ERR_BAD_ARG;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return HB_ERR_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return HB_ERR_CUDA;
  if (prop.major != 10) return HB_ERR_UNSUPPORTED;  // tcgen05 / TMEM kernels: sm_100 only
  const Layout lay = make_layout(*cfg, max_tokens, max_segs, max_page_ids);
  hb_ctx* c = new (std::nothrow) hb_ctx();
  CtxExtra* ex = new (std::nothrow) CtxExtra();
  if (!c || !ex) { delete c; delete ex; return HB_ERR_BAD_ARG; }
  ex->lay = lay;
  ex->pitems.reserve(static_cast<size_t>(lay.max_pool_items));
  ex->aitems.reserve(static_cast<size_t>(lay.max_attn_items));
  ex->titems.reserve(static_cast<size_t>(lay.max_attn_items));
  ex->sort_keys.reserve(static_cast<size_t>(lay.max_attn_items));
  ex->vscratch.lrow.resize(static_cast<size_t>(max_segs));
  ex->vscratch.erow.resize(static_cast<size_t>(max_segs));
  c->cfg = *cfg;
  c->max_tokens = max_tokens;
  c->max_segs = max_segs;
  c->max_page_ids = max_page_ids;
  c->num_sms = prop.multiProcessorCount;
  c->device = dev;
  c->extra = ex;
  c->lm_key = nullptr;
  c->last_launches = 0;
  c->pdl = false;
  if (workspace) {
    if (workspace_bytes < lay.total || (reinterpret_cast<uintptr_t>(workspace) & 255u)) {
      delete c; delete ex;
      return HB_ERR_BAD_ARG;
    }
    c->ws = static_cast<uint8_t*>(workspace);
    c->owns_ws = false;
  } else {
    void* p = nullptr;
    if (cudaMalloc(&p, lay.total) != cudaSuccess) { delete c; delete ex; return HB_ERR_CUDA; }
    c->ws = static_cast<uint8_t*>(p);
    c->owns_ws = true;
  }
  c->ws_bytes = lay.total;
  c->x = reinterpret_cast<float*>(c->ws + lay.x);
  c->h = reinterpret_cast<__half*>(c->ws + lay.h);
  c->q = reinterpret_cast<__half*>(c->ws + lay.q);
  c->attn_out = reinterpret_cast<__half*>(c->ws + lay.attn_out);
  c->act = reinterpret_cast<__half*>(c->ws + lay.act);
  c->lora_u = reinterpret_cast<__half*>(c->ws + lay.lora_u);
  c->lora_part = reinterpret_cast<float*>(c->ws + lay.lora_part);
  c->lora_counters = reinterpret_cast<uint32_t*>(c->ws + lay.lora_counters);
  c->n_lora_counters = static_cast<int32_t>((lay.rows_pad / 128) * 2 * 8);
  c->resid_turns = reinterpret_cast<uint32_t*>(c->ws + lay.resid_turns);
  c->n_resid_turns = lay.n_resid_turns;
  c->logit_in = reinterpret_cast<__half*>(c->ws + lay.logit_in);
  c->rope_cos = reinterpret_cast<float*>(c->ws + lay.rope_cos);
  c->rope_sin = reinterpret_cast<float*>(c->ws + lay.rope_sin);
  c->attn_part = reinterpret_cast<float*>(c->ws + lay.attn_part);
  c->pool_part = reinterpret_cast<float*>(c->ws + lay.pool_part);
  c->counters = reinterpret_cast<uint32_t*>(c->ws + lay.counters);
  c->attn_counters = reinterpret_cast<uint32_t*>(c->ws + lay.attn_counters);
  c->status = reinterpret_cast<uint32_t*>(c->ws + lay.status);
  c->desc_dev = c->ws + lay.desc;
  c->desc_cap = lay.desc_cap;
  c->attn_part_floats = lay.attn_part_floats;
  c->pool_part_floats = lay.pool_part_floats;
  c->n_counters = lay.n_counters;
  c->max_logit_rows = lay.logit_rows_pad;
  c->wmaps.resize(cfg->n_layers);
  for (auto& w : c->wmaps) w.key[0] = w.key[1] = w.key[2] = w.key[3] = nullptr;
  c->lmaps.resize(cfg->n_layers);
  for (auto& m : c->lmaps) {
    for (auto& k : m.key) k = nullptr;
    m.rank = 0;
  }

  int rc = HB_OK;
  bool cuda_ok = true;
  // zero the activation buffers once (rows past the batch feed unused accumulator rows)
  cuda_ok &= cudaMemset(c->ws, 0, lay.total) == cudaSuccess;
  // rotary table: angle(p, i) = p * theta^(-2i/Dh), computed in double, stored as float
  {
    const int half = cfg->head_dim / 2;
    std::vector<float> hc(static_cast<size_t>(cfg->max_pos) * half), hs(hc.size());
    for (int i = 0; i < half; ++i) {
      const double inv_freq = pow(static_cast<double>(cfg->rope_theta), -2.0 * i / cfg->head_dim);
      for (int p = 0; p < cfg->max_pos; ++p) {
        const double a = static_cast<double>(p) * inv_freq;
        hc[static_cast<size_t>(p) * half + i] = static_cast<float>(cos(a));
        hs[static_cast<size_t>(p) * half + i] = static_cast<float>(sin(a));
      }
    }
    cuda_ok &= cudaMemcpy(c->rope_cos, hc.data(), hc.size() * 4, cudaMemcpyHostToDevice) == cudaSuccess;
    cuda_ok &= cudaMemcpy(c->rope_sin, hs.data(), hs.size() * 4, cudaMemcpyHostToDevice) == cudaSuccess;
  }
  for (int i = 0; i < N_STAGING; ++i) {
    cuda_ok &= cudaMallocHost(reinterpret_cast<void**>(&ex->ring[i].host), lay.desc_cap) == cudaSuccess;
    cuda_ok &= cudaEventCreateWithFlags(&ex->ring[i].ev, cudaEventDisableTiming) == cudaSuccess;
  }
  if (cuda_ok) {
    const uint64_t n_q = static_cast<uint64_t>(cfg->n_heads) * cfg->head_dim;
    rc = hb_tmap_2d_f16(&c->tm_h, c->h, lay.rows_pad, cfg->d_model, 128);
    if (rc == HB_OK) rc = hb_tmap_2d_f16(&c->tm_attn_out, c->attn_out, lay.rows_pad, n_q, 128);
    if (rc == HB_OK) rc = hb_tmap_2d_f16(&c->tm_act, c->act, lay.rows_pad, cfg->d_ffn, 128);
    if (rc == HB_OK) rc = hb_tmap_2d_f16(&c->tm_logit_in, c->logit_in, lay.logit_rows_pad, 2ull * cfg->d_model, 128);
    if (rc == HB_OK) rc = hb_tmap_2d_f16(&c->tm_lora_u, c->lora_u, lay.rows_pad, HB_LORA_U_COLS, 128);
  }
  cuda_ok &= cudaDeviceSynchronize() == cudaSuccess;
  if (!cuda_ok || rc != HB_OK) {
    hb_destroy(c);
    return cuda_ok ? rc : HB_ERR_CUDA;
  }
  *out = c;
  return HB_OK;
}

int hb_destroy(hb_ctx* c) {
  if (!c) return HB_ERR_BAD_ARG;
  cudaDeviceSynchronize();
  CtxExtra* ex = extra_of(c);
  if (ex) {
    for (int i = 0; i < N_STAGING; ++i) {
      if (ex->ring[i].host) cudaFreeHost(ex->ring[i].host);
      if (ex->ring[i].ev) cudaEventDestroy(ex->ring[i].ev);
    }
    for (auto* v : {&ex->free_recs, &ex->used_recs})
      for (ProfRec& r : *v) {
        cudaEventDestroy(r.a);
        cudaEventDestroy(r.b);
      }
    delete ex;
  }
  if (c->owns_ws && c->ws) cudaFree(c->ws);
  delete c;
  return HB_OK;
}

// ---- KV pages ----------------------------------------------------------------

int hb_kv_arena_bytes(const hb_model_cfg* cfg, int32_t n_pages, size_t* out_bytes) {
  if (!cfg_ok(cfg) || n_pages < 1 || !out_bytes) return HB_ERR_BAD_ARG;
  *out_bytes = static_cast<size_t>(cfg->n_layers) * n_pages * 2 * cfg->n_kv_heads * cfg->page_size * cfg->head_dim * 2;
  return HB_OK;
}

int hb_kv_create(const hb_model_cfg* cfg, void* arena, size_t arena_bytes, int32_t n_pages, hb_kv** out) {
  if (!out) return HB_ERR_BAD_ARG;
  *out = nullptr;
  size_t need = 0;
  if (hb_kv_arena_bytes(cfg, n_pages, &need) != HB_OK) return HB_ERR_BAD_ARG;
  if (arena && (arena_bytes < need || (reinterpret_cast<uintptr_t>(arena) & 255u))) return HB_ERR_BAD_ARG;
  hb_kv* kv = new (std::nothrow) hb_kv();
  if (!kv) return HB_ERR_BAD_ARG;
  kv->cfg = *cfg;
  kv->has_map = false;
  if (arena) {
    // arena as rows of 64 elements; one copy box = the K+V block of one (page, kv head)
    const uint64_t halves = cfg->head_dim / 64;
    const uint64_t rows = static_cast<uint64_t>(cfg->n_layers) * n_pages * cfg->n_kv_heads * 2 * halves * cfg->page_size;
    if (rows > 0x7fffffffull ||
        hb_tmap_2d_f16(&kv->map, arena, rows, 64, static_cast<uint32_t>(2 * halves * cfg->page_size)) != HB_OK) {
      delete kv;
      return rows > 0x7fffffffull ? HB_ERR_TOO_LARGE : HB_ERR_CUDA;
    }
    kv->has_map = true;
  }
  kv->arena = arena;
  kv->arena_bytes = arena_bytes;
  kv->n_pages = n_pages;
  kv->used.assign(n_pages, 0);
  kv->n_free = n_pages;
  *out = kv;
  return HB_OK;
}

int hb_kv_destroy(hb_kv* kv) {
  if (!kv) return HB_ERR_BAD_ARG;
  delete kv;
  return HB_OK;
}

int hb_kv_alloc_pages(hb_kv* kv, int32_t n, int32_t* out_ids) {
  if (!kv || n < 0 || (n > 0 && !out_ids)) return HB_ERR_BAD_ARG;
  if (n > kv->n_free) return HB_ERR_OOM_PAGES;
  int32_t got = 0;
  for (int32_t p = 0; p < kv->n_pages && got < n; ++p)
    if (!kv->used[p]) {
      kv->used[p] = 1;
      out_ids[got++] = p;
    }
  kv->n_free -= n;
  return HB_OK;
}

int hb_kv_free_pages(hb_kv* kv, int32_t n, const int32_t* ids) {
  if (!kv || n < 0 || (n > 0 && !ids)) return HB_ERR_BAD_ARG;
  for (int32_t i = 0; i < n; ++i) {
    if (ids[i] < 0 || ids[i] >= kv->n_pages || !kv->used[ids[i]]) return HB_ERR_BAD_ARG;
    for (int32_t j = 0; j < i; ++j)
      if (ids[j] == ids[i]) return HB_ERR_BAD_ARG;
  }
  for (int32_t i = 0; i < n; ++i) kv->used[ids[i]] = 0;
  kv->n_free += n;
  return HB_OK;
}

int hb_kv_free_count(const hb_kv* kv, int32_t* out_free) {
  if (!kv || !out_free) return HB_ERR_BAD_ARG;
  *out_free = kv->n_free;
  return HB_OK;
}

// ---- pool slots ----------------------------------------------------------------

int hb_pool_arena_bytes(const hb_model_cfg* cfg, int32_t n_slots, size_t* out_bytes) {
  if (!cfg_ok(cfg) || n_slots < 1 || !out_bytes) return HB_ERR_BAD_ARG;
  *out_bytes = static_cast<size_t>(n_slots) * cfg->d_model * 4 + static_cast<size_t>(n_slots) * 16;
  return HB_OK;
}

int hb_pool_create(const hb_model_cfg* cfg, void* arena, size_t arena_bytes, int32_t n_slots, hb_pool** out) {
  if (!out) return HB_ERR_BAD_ARG;
  *out = nullptr;
  size_t need = 0;
  if (hb_pool_arena_bytes(cfg, n_slots, &need) != HB_OK) return HB_ERR_BAD_ARG;
  if (arena && (arena_bytes < need || (reinterpret_cast<uintptr_t>(arena) & 255u))) return HB_ERR_BAD_ARG;
  hb_pool* p = new (std::nothrow) hb_pool();
  if (!p) return HB_ERR_BAD_ARG;
  p->cfg = *cfg;
  p->arena = arena;
  p->arena_bytes = arena_bytes;
  p->n_slots = n_slots;
  p->used.assign(n_slots, 0);
  p->n_free = n_slots;
  *out = p;
  return HB_OK;
}

int hb_pool_destroy(hb_pool* p) {
  if (!p) return HB_ERR_BAD_ARG;
  delete p;
  return HB_OK;
}

int hb_pool_row_buffer_bytes(const hb_model_cfg* cfg, int32_t n_slots, int32_t max_rows, size_t* out_bytes) {
  if (!cfg_ok(cfg) || n_slots < 1 || max_rows < 1 || max_rows > cfg->max_pos || !out_bytes) return HB_ERR_BAD_ARG;
  *out_bytes = static_cast<size_t>(n_slots) * max_rows * cfg->d_model * 4;
  return HB_OK;
}

int hb_pool_attach_row_buffer(hb_pool* p, void* buf, size_t bytes, int32_t max_rows) {
  if (!p || !buf) return HB_ERR_BAD_ARG;
  size_t need = 0;
  if (hb_pool_row_buffer_bytes(&p->cfg, p->n_slots, max_rows, &need) != HB_OK) return HB_ERR_BAD_ARG;
  if (bytes < need || (reinterpret_cast<uintptr_t>(buf) & 255u)) return HB_ERR_BAD_ARG;
  p->rowbuf = static_cast<float*>(buf);
  p->rowbuf_rows = max_rows;
  return HB_OK;
}

int hb_pool_alloc_slot(hb_pool* p, int32_t* out_slot) {
  if (!p || !out_slot) return HB_ERR_BAD_ARG;
  if (p->n_free == 0) return HB_ERR_OOM_SLOTS;
  for (int32_t s = 0; s < p->n_slots; ++s)
    if (!p->used[s]) {
      p->used[s] = 1;
      --p->n_free;
      *out_slot = s;
      return HB_OK;
    }
  return HB_ERR_OOM_SLOTS;
}

int hb_pool_free_slot(hb_pool* p, int32_t slot) {
  if (!p || slot < 0 || slot >= p->n_slots || !p->used[slot]) return HB_ERR_BAD_ARG;
  p->used[slot] = 0;
  ++p->n_free;
  return HB_OK;
}

// ---- the step --------------------------------------------------------------------

int hb_validate_desc(const hb_model_cfg* cfg, int32_t max_tokens, int32_t max_segs, int32_t max_page_ids,
                     int32_t n_pages, int32_t n_slots, const hb_batch_desc* desc) {
  if (!cfg_ok(cfg)) return HB_ERR_BAD_ARG;
  ValidateScratch vs;   // a stand-alone check has no context to keep its marks in
  return validate(*cfg, max_tokens, max_segs, max_page_ids, n_pages, n_slots, cfg->max_pos, desc, vs);
}

int hb_mixed_step(hb_ctx* c, const hb_batch_desc* d, const hb_weights* w, hb_kv* kv, hb_pool* pool,
                  float* out_logits, float* out_emb, void* stream) {
  return hb_mixed_step_lora(c, d, w, nullptr, kv, pool, out_logits, out_emb, stream);
}

int hb_mixed_step_lora(hb_ctx* c, const hb_batch_desc* d, const hb_weights* w, const hb_lora* lora, hb_kv* kv,
                       hb_pool* pool, float* out_logits, float* out_emb, void* stream) {
  if (!c || !d || !w || !kv || !w->layers || !w->tok_emb || !w->final_norm) return HB_ERR_BAD_ARG;
  if (lora && (lora->rank < 1 || lora->rank > HB_LORA_MAX_RANK || !lora->layers || !(lora->scale == lora->scale)))
    return HB_ERR_BAD_ARG;
  if (!kv->arena || !kv->has_map) return HB_ERR_BAD_ARG;
  if (memcmp(&kv->cfg, &c->cfg, sizeof(hb_model_cfg)) != 0) return HB_ERR_BAD_ARG;
  const int32_t n_slots = pool ? pool->n_slots : 0;
  int rc = validate(c->cfg, c->max_tokens, c->max_segs, c->max_page_ids, kv->n_pages, n_slots,
                    pool ? pool->rowbuf_rows : 0, d, extra_of(c)->vscratch);
  if (rc != HB_OK) return rc;
  if (d->n_logit_rows > 0 && (!out_logits || !w->lm_head)) return HB_ERR_BAD_ARG;
  if (d->n_emb_rows > 0 && !out_emb) return HB_ERR_BAD_ARG;
  // the kernels read and write these with 16-byte (gains: 8-byte) vectors
  if (misaligned(out_logits, 16) || misaligned(out_emb, 16) || misaligned(w->tok_emb, 16) ||
      misaligned(w->final_norm, 8))
    return HB_ERR_BAD_ARG;
  bool any_embed = false;
  for (int32_t r = 0; r < d->n_segs; ++r) any_embed |= (d->segs[r].kind == HB_KIND_EMBED_CHUNK);
  if (any_embed && (!pool || !pool->arena)) return HB_ERR_BAD_ARG;
  c->last_launches = 0;
  if (d->n_tokens == 0) return HB_OK;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const hb_model_cfg& cfg = c->cfg;
  CtxExtra* ex = extra_of(c);

  // ---- pack the descriptor into pinned staging, one H2D copy ----
  Staging& st = ex->ring[ex->next];
  ex->next = (ex->next + 1) % N_STAGING;
  if (st.pending) {
    if (cudaEventSynchronize(st.ev) != cudaSuccess) return HB_ERR_CUDA;
    st.pending = false;
  }
  const int32_t T = d->n_tokens, R = d->n_segs;
  size_t off = 0;
  auto place = [&](size_t bytes) {
    const size_t o = off;
    off = align_up(off + bytes, 16);
    return o;
  };
  const size_t o_tok = place(static_cast<size_t>(T) * 4), o_rseg = place(static_cast<size_t>(T) * 4),
               o_rpos = place(static_cast<size_t>(T) * 4), o_rpage = place(static_cast<size_t>(T) * 4),
               o_segs = place(static_cast<size_t>(R) * sizeof(hb_seg)),
               o_pages = place(static_cast<size_t>(d->n_page_ids) * 4),
               o_lsrc = place(static_cast<size_t>(d->n_logit_rows) * 4);
  int32_t* tok = reinterpret_cast<int32_t*>(st.host + o_tok);
  int32_t* rseg = reinterpret_cast<int32_t*>(st.host + o_rseg);
  int32_t* rpos = reinterpret_cast<int32_t*>(st.host + o_rpos);
  int32_t* rpage = reinterpret_cast<int32_t*>(st.host + o_rpage);
  hb_seg* segs = reinterpret_cast<hb_seg*>(st.host + o_segs);
  int32_t* pages = reinterpret_cast<int32_t*>(st.host + o_pages);
  int32_t* lsrc = reinterpret_cast<int32_t*>(st.host + o_lsrc);
  memcpy(tok, d->token_ids, static_cast<size_t>(T) * 4);
  memcpy(segs, d->segs, static_cast<size_t>(R) * sizeof(hb_seg));
  if (d->n_page_ids) memcpy(pages, d->page_ids, static_cast<size_t>(d->n_page_ids) * 4);
  std::vector<PoolItem>& pitems = ex->pitems;
  pitems.clear();
  int32_t part_at = 0;
  for (int32_t r = 0; r < R; ++r) {
    const hb_seg& sg = d->segs[r];
    for (int32_t j = 0; j < sg.q_len; ++j) {
      rseg[sg.q_start + j] = r;
      rpos[sg.q_start + j] = sg.pos_start + j;
      rpage[sg.q_start + j] = d->page_ids[sg.pt_start + (sg.pos_start + j) / cfg.page_size];
    }
    if (sg.logits_row >= 0) lsrc[sg.logits_row] = sg.q_start + sg.q_len - 1;
    if (sg.kind == HB_KIND_EMBED_CHUNK) {
      if (sg.pool_mode == HB_POOL_MEAN || sg.pool_mode == HB_POOL_WMEAN || sg.pool_mode == HB_POOL_MAX) {
        const int32_t nb = (sg.q_len + POOL_ROWS - 1) / POOL_ROWS;
        for (int32_t b = 0; b < nb; ++b) {
          PoolItem it{};
          it.seg = r;
          it.row0 = sg.q_start + b * POOL_ROWS;
          it.n_rows = std::min(POOL_ROWS, sg.q_len - b * POOL_ROWS);
          it.block = b;
          it.n_blocks = nb;
          it.part_base = part_at;
          pitems.push_back(it);
        }
        part_at += nb;
      } else {  // positional heads: CLS reads the first row of the first chunk, last-token the last row of the final one
        PoolItem it{};
        it.seg = r;
        const bool cls = (sg.pool_mode == HB_POOL_CLS);
        it.row0 = cls ? sg.q_start : sg.q_start + sg.q_len - 1;
        it.n_rows = cls ? (sg.pos_start == 0 ? 1 : 0) : (sg.is_final ? 1 : 0);
        it.block = 0;
        it.n_blocks = 1;
        it.part_base = part_at;
        pitems.push_back(it);
        part_at += 1;
      }
    }
  }
  if (static_cast<int32_t>(pitems.size()) > ex->lay.max_pool_items) return HB_ERR_TOO_LARGE;
  // attention work list: chunk tiles (up to 128 query rows x all visible keys) and decode items (one
  // split of about split_keys keys); sorted by cost, largest first, so the tail of the launch is short
  std::vector<AttnItem>& aitems = ex->aitems;
  std::vector<AttnItem>& titems = ex->titems;
  aitems.clear();
  titems.clear();
  {
    const int G = cfg.n_heads / cfg.n_kv_heads;
    int32_t rec_at = 0;
    for (int32_t r = 0; r < R; ++r) {
      const hb_seg& sg = d->segs[r];
      for (int32_t hk = 0; hk < cfg.n_kv_heads; ++hk) {
        if (sg.kind == HB_KIND_DECODE) {
          const int32_t n_keys = sg.pos_start + 1;
          // about split_keys keys per split, equal parts rounded up to whole 64-key tiles
          const int32_t split_keys = ex->lay.split_keys;
          const int32_t ns0 = std::max(1, (n_keys + split_keys / 2) / split_keys);
          const int32_t per = ((n_keys + ns0 - 1) / ns0 + 63) / 64 * 64;
          const int32_t ns = (n_keys + per - 1) / per;
          for (int32_t sp = 0; sp < ns; ++sp) {
            AttnItem it{};
            it.seg = r; it.kv_head = hk; it.row0 = 0; it.n_rows = G;
            it.key0 = sp * per;
            it.key1 = std::min(n_keys, it.key0 + per);
            it.split = sp; it.n_splits = ns; it.part_base = rec_at; it.mode = 1;
            it.q_start = sg.q_start; it.pos_start = sg.pos_start; it.pt_start = sg.pt_start; it.pt_len = sg.pt_len;
            aitems.push_back(it);
          }
          rec_at += ns;
        } else {
          // chunk rows: tiles of up to 128 rows, all for the tcgen05 body (a short remainder tile costs
          // it less per key tile than it cost the mma.sync body, and that body, left with decode items
          // only, needs fewer registers)
          const int32_t rows = sg.q_len * G;
          for (int32_t row0 = 0; row0 < rows; row0 += ATT_TC_ROWS) {
            AttnItem it{};
            it.seg = r; it.kv_head = hk; it.row0 = row0; it.n_rows = std::min(ATT_TC_ROWS, rows - row0);
            it.key0 = 0;
            it.key1 = sg.pos_start + (row0 + it.n_rows - 1) / G + 1;
            it.split = 0; it.n_splits = 1; it.part_base = 0; it.mode = 0;
            it.q_start = sg.q_start; it.pos_start = sg.pos_start; it.pt_start = sg.pt_start; it.pt_len = sg.pt_len;
            titems.push_back(it);
          }
        }
      }
    }
    if (static_cast<int32_t>(aitems.size() + titems.size()) > ex->lay.max_attn_items) return HB_ERR_TOO_LARGE;
    if (static_cast<size_t>(rec_at) * G * (cfg.head_dim + 2) > c->attn_part_floats) return HB_ERR_TOO_LARGE;
  }
  // Both lists go to the device sorted by cost, largest first (equal costs in list order).  The sort
  // runs over (cost, index) keys in a vector the context owns (std::sort works in place), and the
  // items are copied into the staging buffer in that order.
  // (a tensor-core tile costs its 128 rows whatever part of them is filled)
  auto sorted_into = [&](const std::vector<AttnItem>& items, uint8_t* dst, bool full_tiles) {
    std::vector<uint64_t>& keys = ex->sort_keys;
    keys.clear();
    for (size_t i = 0; i < items.size(); ++i) {
      const AttnItem& a = items[i];
      const uint64_t cost = static_cast<uint64_t>(a.key1 - a.key0) *
                            static_cast<uint64_t>(full_tiles ? ATT_TC_ROWS : (a.mode ? 16 : a.n_rows));
      keys.push_back(((0xffffffffull - std::min<uint64_t>(cost, 0xffffffffull)) << 32) | static_cast<uint64_t>(i));
    }
    std::sort(keys.begin(), keys.end());
    AttnItem* out = reinterpret_cast<AttnItem*>(dst);
    for (size_t i = 0; i < keys.size(); ++i) out[i] = items[static_cast<size_t>(keys[i] & 0xffffffffull)];
  };
  const size_t o_aitems = place(aitems.size() * sizeof(AttnItem));
  const size_t o_titems = place(titems.size() * sizeof(AttnItem));
  const size_t o_pitems = place(pitems.size() * sizeof(PoolItem));
  if (off > c->desc_cap) return HB_ERR_TOO_LARGE;
  if (!pitems.empty()) memcpy(st.host + o_pitems, pitems.data(), pitems.size() * sizeof(PoolItem));
  sorted_into(aitems, st.host + o_aitems, false);
  sorted_into(titems, st.host + o_titems, true);
  if (cudaMemcpyAsync(c->desc_dev, st.host, off, cudaMemcpyHostToDevice, s) != cudaSuccess) return HB_ERR_CUDA;
  if (cudaEventRecord(st.ev, s) != cudaSuccess) return HB_ERR_CUDA;
  st.pending = true;

  DeviceDesc& dd = c->dd;
  dd.tok = reinterpret_cast<const int32_t*>(c->desc_dev + o_tok);
  dd.row_seg = reinterpret_cast<const int32_t*>(c->desc_dev + o_rseg);
  dd.row_pos = reinterpret_cast<const int32_t*>(c->desc_dev + o_rpos);
  dd.row_page = reinterpret_cast<const int32_t*>(c->desc_dev + o_rpage);
  dd.segs = reinterpret_cast<const hb_seg*>(c->desc_dev + o_segs);
  dd.pages = reinterpret_cast<const int32_t*>(c->desc_dev + o_pages);
  dd.logit_src = reinterpret_cast<const int32_t*>(c->desc_dev + o_lsrc);
  dd.attn_items = reinterpret_cast<const AttnItem*>(c->desc_dev + o_aitems);
  dd.tc_items = reinterpret_cast<const AttnItem*>(c->desc_dev + o_titems);
  dd.pool_items = reinterpret_cast<const PoolItem*>(c->desc_dev + o_pitems);
  dd.T = T;
  dd.R = R;
  dd.n_logit = d->n_logit_rows;
  dd.n_attn_items = static_cast<int32_t>(aitems.size());
  dd.n_tc_items = static_cast<int32_t>(titems.size());
  dd.n_pool_items = static_cast<int32_t>(pitems.size());

  KvGeom kg;
  kg.arena = static_cast<__half*>(kv->arena);
  kg.Hkv = cfg.n_kv_heads;
  kg.P = cfg.page_size;
  kg.Dh = cfg.head_dim;
  kg.n_pages = kv->n_pages;
  kg.page_stride = 2ll * cfg.n_kv_heads * cfg.page_size * cfg.head_dim;
  kg.layer_stride = kg.page_stride * kv->n_pages;

  const int n_qkv = (cfg.n_heads + 2 * cfg.n_kv_heads) * cfg.head_dim;
  const int n_q = cfg.n_heads * cfg.head_dim;
  // adapters apply to EMBED_CHUNK rows, which are the last rows of the batch (kinds are sorted)
  int32_t first_embed_row = T;
  for (int32_t r = 0; r < R; ++r)
    if (d->segs[r].kind == HB_KIND_EMBED_CHUNK) { first_embed_row = d->segs[r].q_start; break; }
  const bool use_lora = (lora != nullptr) && first_embed_row < T;
  const int r1 = 64, r2 = use_lora ? (2 * lora->rank + 63) / 64 * 64 : 0, r3 = use_lora ? (3 * lora->rank + 63) / 64 * 64 : 0;
  int launches = 0;
  // Kernels after the first may become resident while their predecessor drains (programmatic
  // dependent launch); not while per-launch events are being recorded between them.
  const bool pdl_enabled = !ex->profiling;
  c->pdl = false;
  auto prof_begin = [&](int cls) -> ProfRec* {
    if (!ex->profiling) return nullptr;
    ProfRec r;
    if (!ex->free_recs.empty()) {
      r = ex->free_recs.back();
      ex->free_recs.pop_back();
    } else if (cudaEventCreate(&r.a) != cudaSuccess || cudaEventCreate(&r.b) != cudaSuccess) {
      return nullptr;
    }
    r.cls = cls;
    cudaEventRecord(r.a, s);
    ex->used_recs.push_back(r);
    return &ex->used_recs.back();
  };
  auto prof_end = [&](ProfRec* r) {
    if (r) cudaEventRecord(r->b, s);
  };
#define HB_TRY(cls, expr)             \
  do {                                \
    ProfRec* pr__ = prof_begin(cls);  \
    const int rc__ = (expr);          \
    prof_end(pr__);                   \
    if (rc__ != HB_OK) return rc__;   \
    ++launches;                       \
    c->pdl = pdl_enabled;             \
  } while (0)

  for (int l = 0; l < cfg.n_layers; ++l) {
    const hb_layer_weights& lw = w->layers[l];
    if (!lw.attn_norm || !lw.wqkv || !lw.wo || !lw.ffn_norm || !lw.w_gate_up || !lw.w_down) return HB_ERR_BAD_ARG;
    if (misaligned(lw.attn_norm, 8) || misaligned(lw.ffn_norm, 8)) return HB_ERR_BAD_ARG;
    hb_ctx::WMaps& wm = c->wmaps[l];
    if (wm.key[0] != lw.wqkv || wm.key[1] != lw.wo || wm.key[2] != lw.w_gate_up || wm.key[3] != lw.w_down) {
      wm.bn_qkv = hb_gemm_pick_bn(c->max_tokens, n_qkv, c->num_sms);
      wm.bn_o = hb_gemm_pick_bn(c->max_tokens, cfg.d_model, c->num_sms);
      wm.bn_gu = hb_gemm_pick_bn(c->max_tokens, 2 * cfg.d_ffn, c->num_sms);
      wm.bn_down = wm.bn_o;
      wm.ks_o = hb_gemm_pick_ksplit(c->max_tokens, cfg.d_model, n_q, wm.bn_o, c->num_sms);
      wm.ks_down = hb_gemm_pick_ksplit(c->max_tokens, cfg.d_model, cfg.d_ffn, wm.bn_down, c->num_sms);
      if ((rc = hb_tmap_2d_f16(&wm.qkv, lw.wqkv, n_qkv, cfg.d_model, hb_gemm_box_rows(wm.bn_qkv))) != HB_OK) return rc;
      if ((rc = hb_tmap_2d_f16(&wm.o, lw.wo, cfg.d_model, n_q, hb_gemm_box_rows(wm.bn_o))) != HB_OK) return rc;
      if ((rc = hb_tmap_2d_f16(&wm.gu, lw.w_gate_up, 2ull * cfg.d_ffn, cfg.d_model, hb_gemm_box_rows(wm.bn_gu))) != HB_OK) return rc;
      if ((rc = hb_tmap_2d_f16(&wm.down, lw.w_down, cfg.d_model, cfg.d_ffn, hb_gemm_box_rows(wm.bn_down))) != HB_OK) return rc;
      wm.key[0] = lw.wqkv; wm.key[1] = lw.wo; wm.key[2] = lw.w_gate_up; wm.key[3] = lw.w_down;
    }
    // adapters: tensor maps of this layer's packed factors (cached by pointer)
    hb_ctx::LMaps* lm = nullptr;
    if (use_lora) {
      const hb_lora_layer& ll = lora->layers[l];
      const void* keys[8] = {ll.a_qkv, ll.b_qkv, ll.a_o, ll.b_o, ll.a_gu, ll.b_gu, ll.a_d, ll.b_d};
      for (const void* k : keys)
        if (!k) return HB_ERR_BAD_ARG;
      lm = &c->lmaps[l];
      if (lm->rank != lora->rank || memcmp(lm->key, keys, sizeof(keys)) != 0) {
        if ((rc = hb_tmap_2d_f16(&lm->a_qkv, ll.a_qkv, r3, cfg.d_model, r3 > 128 ? 256 : 128)) != HB_OK) return rc;
        if ((rc = hb_tmap_2d_f16(&lm->b_qkv, ll.b_qkv, n_qkv, r3, hb_gemm_box_rows(wm.bn_qkv))) != HB_OK) return rc;
        if ((rc = hb_tmap_2d_f16(&lm->a_o, ll.a_o, r1, n_q, 128)) != HB_OK) return rc;
        if ((rc = hb_tmap_2d_f16(&lm->b_o, ll.b_o, cfg.d_model, r1, hb_gemm_box_rows(wm.bn_o))) != HB_OK) return rc;
        if ((rc = hb_tmap_2d_f16(&lm->a_gu, ll.a_gu, r2, cfg.d_model, r2 > 128 ? 256 : 128)) != HB_OK) return rc;
        if ((rc = hb_tmap_2d_f16(&lm->b_gu, ll.b_gu, 2ull * cfg.d_ffn, r2, hb_gemm_box_rows(wm.bn_gu))) != HB_OK) return rc;
        if ((rc = hb_tmap_2d_f16(&lm->a_d, ll.a_d, r1, cfg.d_ffn, 128)) != HB_OK) return rc;
        if ((rc = hb_tmap_2d_f16(&lm->b_d, ll.b_d, cfg.d_model, r1, hb_gemm_box_rows(wm.bn_down))) != HB_OK) return rc;
        memcpy(lm->key, keys, sizeof(keys));
        lm->rank = lora->rank;
      }
    }
    // rank-r activations of the adapted rows for the projection that reads activation map `tmX`
    // with K columns: u = scale * (x A^T), zero for rows before the first embedding row
    auto lora_down = [&](const CUtensorMap& tmX, const CUtensorMap& tmAfac, int R, int K) -> int {
      GemmArgs gu = {};
      gu.status = c->status;
      gu.M = T; gu.N = R; gu.K = K; gu.C = c->lora_u; gu.ldc = HB_LORA_U_COLS;
      gu.alpha = lora->scale; gu.first_row = first_embed_row;
      // split K four ways (fewer when K is short): the split depends on K alone, so a row's
      // summation order is the same in every batch
      gu.k_splits = std::min(HB_LORA_K_SPLITS, (K + 63) / 64);
      gu.split_part = c->lora_part; gu.split_counters = c->lora_counters;
      return hb_gemm_launch(tmX, tmAfac, R > 128 ? 256 : 128, HB_EPI_LORA_DOWN, gu, c->num_sms, s, nullptr, nullptr,
                            c->pdl);
    };
    if (l == 0) HB_TRY(HB_CLASS_NORM_ROPE, hb_launch_embed_norm(c, w->tok_emb, lw.attn_norm, s));
    else HB_TRY(HB_CLASS_NORM_ROPE, hb_launch_rmsnorm(c, lw.attn_norm, s));
    GemmArgs ga = {};
    ga.status = c->status;
    ga.b_kshift = 0;
    ga.M = T;
    // tile variant of this step's launches (the maps serve both; see hb_gemm_pick_step_variant)
    const int kb_d = (cfg.d_model + 63) / 64, kb_q = (n_q + 63) / 64, kb_f = (cfg.d_ffn + 63) / 64;
    const int v_qkv = hb_gemm_pick_step_variant(wm.bn_qkv, T, n_qkv, kb_d + (use_lora ? r3 / 64 : 0), 1, c->num_sms);
    const int v_o = hb_gemm_pick_step_variant(wm.bn_o, T, cfg.d_model, kb_q + (use_lora ? r1 / 64 : 0), wm.ks_o, c->num_sms);
    const int v_gu = hb_gemm_pick_step_variant(wm.bn_gu, T, 2 * cfg.d_ffn, kb_d + (use_lora ? r2 / 64 : 0), 1, c->num_sms);
    const int v_down = hb_gemm_pick_step_variant(wm.bn_down, T, cfg.d_model, kb_f + (use_lora ? r1 / 64 : 0), wm.ks_down, c->num_sms);
    // QKV projection; its epilogue rotates q, k and appends k, v to the pages
    ga.C = nullptr; ga.N = n_qkv; ga.K = cfg.d_model; ga.ldc = n_qkv;
    ga.row_pos = dd.row_pos; ga.row_page = dd.row_page; ga.rope_cos = c->rope_cos; ga.rope_sin = c->rope_sin;
    ga.q_out = c->q; ga.kv_layer = kg.arena + static_cast<int64_t>(l) * kg.layer_stride;
    ga.page_stride = kg.page_stride; ga.Hq = cfg.n_heads; ga.Hkv = cfg.n_kv_heads; ga.Dh = cfg.head_dim;
    ga.P = cfg.page_size; ga.n_pages = kg.n_pages;
    if (use_lora) HB_TRY(HB_CLASS_LORA, lora_down(c->tm_h, lm->a_qkv, r3, cfg.d_model));
    ga.k2_blocks = use_lora ? r3 / 64 : 0;
    HB_TRY(HB_CLASS_GEMM, hb_gemm_launch(c->tm_h, wm.qkv, v_qkv, HB_EPI_QKV_ROPE, ga, c->num_sms, s,
                                         use_lora ? &c->tm_lora_u : nullptr, use_lora ? &lm->b_qkv : nullptr, c->pdl));
    if (ex->profiling) {
      // timed per class: one launch per item list (the same kernel over one list)
      if (dd.n_tc_items > 0)
        HB_TRY(HB_CLASS_ATTENTION_TC, hb_launch_attention(c, kg, kv->map, l, s, HB_ATTN_CHUNK_TILES));
      if (dd.n_attn_items > 0)
        HB_TRY(HB_CLASS_ATTENTION, hb_launch_attention(c, kg, kv->map, l, s, HB_ATTN_SMALL_ITEMS));
    } else if (dd.n_tc_items + dd.n_attn_items > 0) {
      HB_TRY(HB_CLASS_ATTENTION, hb_launch_attention(c, kg, kv->map, l, s, HB_ATTN_ALL));
    }
    // O projection, added to the residual stream
    ga.C = c->x; ga.N = cfg.d_model; ga.K = n_q; ga.ldc = cfg.d_model;
    ga.k_splits = wm.ks_o; ga.split_counters = c->resid_turns;
    if (use_lora) HB_TRY(HB_CLASS_LORA, lora_down(c->tm_attn_out, lm->a_o, r1, n_q));
    ga.k2_blocks = use_lora ? r1 / 64 : 0;
    HB_TRY(HB_CLASS_GEMM, hb_gemm_launch(c->tm_attn_out, wm.o, v_o, HB_EPI_RESID_F32, ga, c->num_sms, s,
                                         use_lora ? &c->tm_lora_u : nullptr, use_lora ? &lm->b_o : nullptr, c->pdl));
    HB_TRY(HB_CLASS_NORM_ROPE, hb_launch_rmsnorm(c, lw.ffn_norm, s));
    // gate/up projection with SwiGLU
    ga.C = c->act; ga.N = 2 * cfg.d_ffn; ga.K = cfg.d_model; ga.ldc = cfg.d_ffn;
    ga.k_splits = 1;
    if (use_lora) HB_TRY(HB_CLASS_LORA, lora_down(c->tm_h, lm->a_gu, r2, cfg.d_model));
    ga.k2_blocks = use_lora ? r2 / 64 : 0;
    HB_TRY(HB_CLASS_GEMM, hb_gemm_launch(c->tm_h, wm.gu, v_gu, HB_EPI_SWIGLU, ga, c->num_sms, s,
                                         use_lora ? &c->tm_lora_u : nullptr, use_lora ? &lm->b_gu : nullptr, c->pdl));
    // down projection, added to the residual stream
    ga.C = c->x; ga.N = cfg.d_model; ga.K = cfg.d_ffn; ga.ldc = cfg.d_model;
    ga.k_splits = wm.ks_down; ga.split_counters = c->resid_turns;
    if (use_lora) HB_TRY(HB_CLASS_LORA, lora_down(c->tm_act, lm->a_d, r1, cfg.d_ffn));
    ga.k2_blocks = use_lora ? r1 / 64 : 0;
    HB_TRY(HB_CLASS_GEMM, hb_gemm_launch(c->tm_act, wm.down, v_down, HB_EPI_RESID_F32, ga, c->num_sms, s,
                                         use_lora ? &c->tm_lora_u : nullptr, use_lora ? &lm->b_d : nullptr, c->pdl));
  }
  float* pool_sum = pool ? static_cast<float*>(pool->arena) : nullptr;
  uint32_t* pool_meta = pool ? reinterpret_cast<uint32_t*>(static_cast<uint8_t*>(pool->arena) +
                                                           static_cast<size_t>(pool->n_slots) * cfg.d_model * 4)
                             : nullptr;
  {
    ProfRec* pr = prof_begin(HB_CLASS_POOL);
    rc = hb_launch_final(c, w->final_norm, pool_sum, pool_meta, n_slots, pool ? pool->rowbuf : nullptr,
                         pool ? pool->rowbuf_rows : 0, out_emb, s);
    prof_end(pr);
    if (rc != HB_OK) return rc;
    launches += (dd.n_logit > 0) + (dd.n_pool_items > 0);
    c->pdl = pdl_enabled;
  }
  if (dd.n_logit > 0) {
    if (c->lm_key != w->lm_head) {
      if ((rc = hb_tmap_2d_f16(&c->tm_lm, w->lm_head, cfg.vocab, cfg.d_model, 128)) != HB_OK) return rc;
      c->lm_key = w->lm_head;
    }
    GemmArgs ga = {};
    ga.status = c->status;
    ga.b_kshift = 1;  // A holds (hi, lo) 64-column blocks: each weight k-block is used twice
    ga.M = dd.n_logit; ga.N = cfg.vocab; ga.K = 2 * cfg.d_model; ga.ldc = cfg.vocab; ga.C = out_logits;
    // a few logits rows stream the weights through single-CTA tiles; hundreds of them (decode-heavy
    // steps) are a real contraction and take the pair tiles (same boxes, same bits)
    const int v_lm = hb_gemm_pick_step_variant(128, dd.n_logit, cfg.vocab, (2 * cfg.d_model + 63) / 64, 1, c->num_sms);
    HB_TRY(HB_CLASS_LM_HEAD, hb_gemm_launch(c->tm_logit_in, c->tm_lm, v_lm, HB_EPI_F32, ga, c->num_sms, s, nullptr,
                                            nullptr, c->pdl));
  }
#undef HB_TRY
  c->last_launches = launches;
  c->pdl = false;
  return HB_OK;
}

int hb_argmax(hb_ctx* c, const float* logits, int32_t n_rows, int32_t* out_tokens, void* stream) {
  if (!c || n_rows < 0 || (n_rows > 0 && (!logits || !out_tokens))) return HB_ERR_BAD_ARG;
  return hb_launch_argmax(logits, n_rows, c->cfg.vocab, out_tokens, static_cast<cudaStream_t>(stream));
}

int hb_weights_pack_f16(const void* src_bf16, void* dst_f16, size_t n_elems, void* stream) {
  if (!src_bf16 || !dst_f16) return HB_ERR_BAD_ARG;
  if ((reinterpret_cast<uintptr_t>(src_bf16) & 15u) || (reinterpret_cast<uintptr_t>(dst_f16) & 15u)) return HB_ERR_BAD_ARG;
  if (src_bf16 != dst_f16) {   // partial overlap would corrupt the input
    const char* a = static_cast<const char*>(src_bf16);
    const char* b = static_cast<const char*>(dst_f16);
    if (a < b + n_elems * 2 && b < a + n_elems * 2) return HB_ERR_BAD_ARG;
  }
  return hb_launch_bf16_to_f16(src_bf16, dst_f16, n_elems, static_cast<cudaStream_t>(stream));
}

int hb_pool_chunk(hb_ctx* c, const float* x, const void* gain, int32_t n_rows, int32_t mode, int32_t first_chunk,
                  int32_t is_final, float* slot_sum, uint32_t* slot_meta, float* out_emb, void* stream) {
  if (!c || !x || !gain || !slot_sum || !slot_meta || n_rows < 1) return HB_ERR_BAD_ARG;
  if (mode < HB_POOL_MEAN || mode > HB_POOL_WMEAN) return HB_ERR_BAD_ARG;
  if (is_final && !out_emb) return HB_ERR_BAD_ARG;
  // 16-byte vector accesses to the rows, the slot and the output; 8-byte ones to the gain
  if (misaligned(x, 16) || misaligned(slot_sum, 16) || misaligned(out_emb, 16) || misaligned(gain, 8) ||
      misaligned(slot_meta, 4))
    return HB_ERR_BAD_ARG;
  if (n_rows > c->max_tokens) return HB_ERR_TOO_LARGE;
  return hb_launch_pool_chunk(c, x, gain, n_rows, mode, first_chunk != 0, is_final != 0, slot_sum, slot_meta,
                              out_emb, static_cast<cudaStream_t>(stream));
}

int hb_selftest_wait_expiry(hb_ctx* c, uint32_t limit_ms, void* stream) {
  if (!c || limit_ms < 1 || limit_ms > 1000) return HB_ERR_BAD_ARG;
  return hb_launch_wait_expiry_selftest(c, static_cast<uint64_t>(limit_ms) * 1000000ull, static_cast<cudaStream_t>(stream));
}

int hb_status_poll(hb_ctx* c, void* stream, uint32_t* out_code) {
  if (!c) return HB_ERR_BAD_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  uint32_t code = 0;
  if (cudaMemcpyAsync(&code, c->status, 4, cudaMemcpyDeviceToHost, s) != cudaSuccess) return HB_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return HB_ERR_CUDA;
  if (code != 0) {
    // a block that gave up may have left arrival counters mid-count: clear them with the status word
    if (cudaMemsetAsync(c->attn_counters, 0, static_cast<size_t>(c->max_segs) * c->cfg.n_kv_heads * 4, s) !=
            cudaSuccess ||
        cudaMemsetAsync(c->counters, 0, static_cast<size_t>(c->n_counters) * 4, s) != cudaSuccess ||
        cudaMemsetAsync(c->lora_counters, 0, static_cast<size_t>(c->n_lora_counters) * 4, s) != cudaSuccess ||
        cudaMemsetAsync(c->resid_turns, 0, static_cast<size_t>(c->n_resid_turns) * 4, s) != cudaSuccess)
      return HB_ERR_CUDA;
    // (the status block also holds the attention kernel's work queue: words 8 and 9)
    if (cudaMemsetAsync(c->status, 0, 64, s) != cudaSuccess) return HB_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return HB_ERR_CUDA;
  }
  if (out_code) *out_code = code;
  return code ? HB_ERR_DEVICE_STATUS : HB_OK;
}

int hb_profile_enable(hb_ctx* c, int on) {
  if (!c) return HB_ERR_BAD_ARG;
  extra_of(c)->profiling = (on != 0);
  return HB_OK;
}

int hb_profile_read(hb_ctx* c, float* ms_by_class, int32_t* launches_by_class) {
  if (!c || !ms_by_class || !launches_by_class) return HB_ERR_BAD_ARG;
  CtxExtra* ex = extra_of(c);
  for (ProfRec& r : ex->used_recs) {
    float ms = 0.f;
    if (cudaEventSynchronize(r.b) != cudaSuccess || cudaEventElapsedTime(&ms, r.a, r.b) != cudaSuccess)
      return HB_ERR_CUDA;
    ms_by_class[r.cls] += ms;
    launches_by_class[r.cls] += 1;
    ex->free_recs.push_back(r);
  }
  ex->used_recs.clear();
  return HB_OK;
}

int hb_last_launch_count(const hb_ctx* c, int32_t* out_count) {
  if (!c || !out_count) return HB_ERR_BAD_ARG;
  *out_count = c->last_launches;
  return HB_OK;
}

int hb_gemm_set_walk(int32_t band, int32_t hints) {
  if (band < -1 || hints < -1 || hints > 1) return HB_ERR_BAD_ARG;
  hb_gemm_walk_override(band, hints);
  return HB_OK;
}

int hb_gemm_set_cta_limit(int32_t max_ctas) {
  if (max_ctas < 0 || (max_ctas & 1)) return HB_ERR_BAD_ARG;
  hb_gemm_cta_limit(max_ctas);
  return HB_OK;
}

int hb_attn_set_split_keys(int32_t keys) {
  if (keys == 0) keys = 2048;
  if (keys < 256 || keys > 65536 || (keys & 63)) return HB_ERR_BAD_ARG;
  g_att_split_keys = keys;
  return HB_OK;
}

int hb_attn_set_block_limit(int32_t max_blocks) {
  if (max_blocks < 0) return HB_ERR_BAD_ARG;
  hb_attn_block_limit(max_blocks);
  return HB_OK;
}

int hb_gemm(hb_ctx* c, const void* A, const void* B, void* C, int32_t M, int32_t N, int32_t K, int32_t epilogue,
            void* stream) {
  return hb_gemm_pair(c, A, B, nullptr, nullptr, C, M, N, K, 0, epilogue, stream);
}

int hb_gemm_pair(hb_ctx* c, const void* A, const void* B, const void* A2, const void* B2, void* C, int32_t M,
                 int32_t N, int32_t K, int32_t K2, int32_t epilogue, void* stream) {
  if (!c || !A || !B || !C || M < 1 || N < 8 || K < 8 || (N & 7) || (K & 7)) return HB_ERR_BAD_ARG;
  if (epilogue < HB_EPI_F16 || epilogue > HB_EPI_SWIGLU) return HB_ERR_BAD_ARG;
  if (epilogue == HB_EPI_SWIGLU && (N & 15)) return HB_ERR_BAD_ARG;
  if (reinterpret_cast<uintptr_t>(C) & 15u) return HB_ERR_BAD_ARG;
  if (K2 < 0 || (K2 & 63) || ((K2 > 0) != (A2 != nullptr && B2 != nullptr))) return HB_ERR_BAD_ARG;
  const int bn = hb_gemm_pick_bn(M, N, c->num_sms);
  CUtensorMap ta, tb, ta2, tb2;
  int rc = hb_tmap_2d_f16(&ta, A, M, K, 128);
  if (rc != HB_OK) return rc;
  rc = hb_tmap_2d_f16(&tb, B, N, K, hb_gemm_box_rows(bn));
  if (rc != HB_OK) return rc;
  if (K2 > 0) {
    if ((rc = hb_tmap_2d_f16(&ta2, A2, M, K2, 128)) != HB_OK) return rc;
    if ((rc = hb_tmap_2d_f16(&tb2, B2, N, K2, hb_gemm_box_rows(bn))) != HB_OK) return rc;
  }
  GemmArgs ga = {};
  ga.C = C; ga.M = M; ga.N = N; ga.K = K; ga.b_kshift = 0; ga.status = c->status;
  ga.k2_blocks = K2 / 64;
  ga.ldc = (epilogue == HB_EPI_SWIGLU) ? N / 2 : N;
  if (epilogue == HB_EPI_RESID_F32) {
    const int ks = hb_gemm_pick_ksplit(M, N, K, bn, c->num_sms);
    const long turns = static_cast<long>((M + 255) / 256) * ((N + 255) / 256) * 2 * 8;
    if (ks > 1 && turns <= c->n_resid_turns) {
      ga.k_splits = ks;
      ga.split_counters = c->resid_turns;
    }
  }
  return hb_gemm_launch(ta, tb, bn, epilogue, ga, c->num_sms, static_cast<cudaStream_t>(stream),
                        K2 > 0 ? &ta2 : nullptr, K2 > 0 ? &tb2 : nullptr);
}

}  // extern "C"
