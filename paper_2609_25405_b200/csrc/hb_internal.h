// Internal declarations shared by the translation units of libhb.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <vector>

#include "../../include/hb.h"

// Words of the status block the attention kernel uses as its work queue (tickets, blocks gone).
constexpr int HB_STATUS_ATTN_QUEUE_WORD = 8;
// Device status codes (OR-ed into the context's status word).
enum : uint32_t {
  HB_DEV_GEMM_WAIT_EXPIRED = 1u << 0,
  HB_DEV_ATTN_BAD_INDEX = 1u << 1,
  HB_DEV_APPEND_BAD_INDEX = 1u << 2,
  HB_DEV_POOL_BAD_INDEX = 1u << 3,
  HB_DEV_ATTN_WAIT_EXPIRED = 1u << 4,
  HB_DEV_SELFTEST_WAIT_EXPIRED = 1u << 5,
  HB_DEV_F16_RANGE = 1u << 6,   // a normed row or a SwiGLU output was NaN or beyond the largest finite half
};

// Attention work item: one (segment, kv head, row tile, key split).
struct AttnItem {
  int32_t seg;        // segment index
  int32_t kv_head;
  int32_t row0;       // first row of the tile inside the segment
  int32_t n_rows;     // rows in the tile
  int32_t key0;       // first key of this split
  int32_t key1;       // one past the last key this split may touch
  int32_t split;      // split index, n_splits
  int32_t n_splits;
  int32_t part_base;  // first partial-result record of this (seg, kv_head)
  int32_t mode;       // 0 = chunk item (query-row tile, all keys), 1 = decode item (one split)
  // copied from the segment so that a CTA needs one load to know its work
  int32_t q_start;    // first token row of the segment
  int32_t pos_start;  // tokens already cached when the segment starts
  int32_t pt_start;   // offset of the request's page list inside the page-id array
  int32_t pt_len;
  int32_t pad[2];
};

// Pool work item: rows [row0, row0 + n_rows) of an embedding segment.
struct PoolItem {
  int32_t seg;
  int32_t row0;       // absolute token row
  int32_t n_rows;
  int32_t block;      // block index inside the segment
  int32_t n_blocks;
  int32_t part_base;  // first partial-sum record of the segment
  int32_t pad[2];
};

struct DeviceDesc {
  // all device pointers into the context's descriptor buffer
  const int32_t* tok;       // [T]
  const int32_t* row_seg;   // [T]
  const int32_t* row_pos;   // [T]
  const int32_t* row_page;  // [T] page holding the row's own position
  const hb_seg* segs;       // [R]
  const int32_t* pages;     // [n_page_ids]
  const int32_t* logit_src; // [n_logit_rows] token row feeding logits row i
  const AttnItem* attn_items;  // decode splits (mma.sync body)
  const AttnItem* tc_items;    // chunk tiles of up to 128 rows (tcgen05 body)
  const PoolItem* pool_items;
  int32_t T, R, n_logit, n_attn_items, n_tc_items, n_pool_items;
};

struct KvGeom {
  __half* arena;
  int64_t layer_stride;  // elements
  int64_t page_stride;   // elements: Hkv * 2 * Dh * P; inside a page: [kv head][K|V][Dh/64][P][64]
  int32_t n_pages, Hkv, P, Dh;
};

struct hb_kv {
  hb_model_cfg cfg;
  CUtensorMap map;      // arena as a 2-D tensor [rows of 64 fp16], box = the K+V block of one (page, kv head)
  bool has_map;
  void* arena;
  size_t arena_bytes;
  int32_t n_pages;
  std::vector<uint8_t> used;
  int32_t n_free;
};

struct hb_pool {
  hb_model_cfg cfg;
  void* arena;
  size_t arena_bytes;
  int32_t n_slots;
  std::vector<uint8_t> used;
  int32_t n_free;
  float* rowbuf = nullptr;    // buffered heads: [n_slots][rowbuf_rows][d] final hidden states, fp32
  int32_t rowbuf_rows = 0;
};

// ---- GEMM -------------------------------------------------------------------
// Internal epilogue of the QKV projection: rotary embedding and KV-page append fused into the
// accumulator read-out (not reachable through hb_gemm).
constexpr int HB_EPI_QKV_ROPE = 4;
// Internal epilogue of the adapters' down projection u = alpha * (x A^T): fp16 out, rows before
// GemmArgs::first_row stored as zero (tile width 128 only).
constexpr int HB_EPI_LORA_DOWN = 5;
constexpr int HB_LORA_K_SPLITS = 4;
constexpr int HB_LORA_MAX_RANK = 64;
constexpr int HB_LORA_U_COLS = 192;   // three rank-64 blocks: the fused q, k, v projection

struct GemmArgs {
  void* C;
  int32_t M, N, K;      // K = columns of A; B has K >> b_kshift columns
  int32_t ldc;          // elements
  int32_t b_kshift;     // B k-block index = A k-block index >> b_kshift
  int32_t k2_blocks;    // 64-column blocks of the second operand pair accumulated after K (0 = none)
  int32_t raster_band;  // row tiles per band of the tile walk (0 = all: rows fastest over the whole M); set by hb_gemm_launch
  int32_t l2_hints;     // 1: A loads are kept in L2 (evict last), B loads stream (evict first); set by hb_gemm_launch
  uint32_t* status;
  // HB_EPI_LORA_DOWN only
  float alpha;
  int32_t first_row;
  // HB_EPI_LORA_DOWN and HB_EPI_RESID_F32
  int32_t k_splits;          // work items per output tile (0 or 1 = no split), each over an equal share of the K blocks
  float* split_part;         // LORA_DOWN: [k_splits, M, N] partial sums (k_splits > 1)
  uint32_t* split_counters;  // LORA_DOWN: [tiles * 8] arrival counters; RESID_F32: [tiles * CG * 8] turn words (one per epilogue warp); zero between launches
  // HB_EPI_QKV_ROPE only
  const int32_t* row_pos;   // [M] position of each row inside its request
  const int32_t* row_page;  // [M] physical page that holds that position
  const float* rope_cos;    // [max_pos, Dh/2]
  const float* rope_sin;
  __half* q_out;            // [M, Hq*Dh]
  __half* kv_layer;         // this layer's slice of the KV arena
  int64_t page_stride;      // elements per page: 2 * Hkv * P * Dh
  int32_t Hq, Hkv, Dh, P, n_pages;
};

// 2-D tensor map over a row-major 16-bit matrix (fp16 everywhere in this library), 64-column boxes,
// 128-byte swizzle.
int hb_tmap_2d_f16(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols,
                   uint32_t box_rows);

// Dynamic shared memory above 48 KiB has to be enabled per kernel ON EVERY DEVICE the kernel runs
// on.  One of these per kernel instantiation remembers, per device, the largest size enabled so
// far; hb_ensure_dyn_smem raises it on the current device when a launch needs more.
constexpr int HB_MAX_DEVICES = 64;
struct DynSmemState {
  std::atomic<int> bytes[HB_MAX_DEVICES];
};
inline int hb_ensure_dyn_smem(const void* kern, DynSmemState& st, int bytes) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= HB_MAX_DEVICES) return HB_ERR_CUDA;
  if (st.bytes[dev].load(std::memory_order_acquire) >= bytes) return HB_OK;
  // two threads may both get here: the attribute call is idempotent
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return HB_ERR_CUDA;
  int seen = st.bytes[dev].load(std::memory_order_relaxed);
  while (seen < bytes && !st.bytes[dev].compare_exchange_weak(seen, bytes, std::memory_order_release)) {}
  return HB_OK;
}
// GEMM variants: 128 / 256 = one CTA per 128 x BN tile; HB_GEMM_PAIR256 = a CTA pair per 256 x 256 tile.
// The B tensor map's box must have hb_gemm_box_rows(variant) rows.
constexpr int HB_GEMM_PAIR256 = 512;
int hb_gemm_pick_bn(int M, int N, int num_sms);
int hb_gemm_box_rows(int variant);
int hb_gemm_pick_ksplit(int M, int N, int K, int variant, int num_sms);
// Variant for one launch of `rows` rows when the B map was built for `map_variant` (the choice made
// for the context's row capacity): a step much smaller than the capacity may run single-CTA tiles.
int hb_gemm_pick_step_variant(int map_variant, int rows, int N, int k_blocks, int k_splits, int num_sms);
// Chooses GemmArgs::raster_band and l2_hints for a launch of `variant` (called by hb_gemm_launch).
void hb_gemm_pick_walk(int variant, int epi, GemmArgs* g);
void hb_gemm_walk_override(int band, int hints);
void hb_attn_block_limit(int max_blocks);   // tests: > 0 caps the resident blocks of every attention launch, 0 = two per SM
void hb_gemm_cta_limit(int max_ctas);   // tuning: > 0 caps the CTAs of every projection launch, 0 = all SMs   // tuning: >= 0 forces the value for every launch, -1 = automatic
int hb_gemm_launch(const CUtensorMap& tmA, const CUtensorMap& tmB, int bn, int epi,
                   const GemmArgs& a, int num_sms, cudaStream_t s, const CUtensorMap* tmA2 = nullptr,
                   const CUtensorMap* tmB2 = nullptr, bool pdl = false);

// Plain launch, optionally allowed to overlap the tail of the previous kernel of the stream (the
// kernel must then start with grid_dep_wait()).
template <typename... KArgs, typename... Args>
inline int hb_launch_kernel(void (*kern)(KArgs...), unsigned grid, unsigned block, size_t smem, cudaStream_t s,
                            bool pdl, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(block);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...) == cudaSuccess ? HB_OK : HB_ERR_CUDA;
}

// ---- elementwise / attention launchers ---------------------------------------
struct hb_ctx;
int hb_launch_embed_norm(hb_ctx* c, const void* tok_emb, const void* gain, cudaStream_t s);
int hb_launch_rmsnorm(hb_ctx* c, const void* gain, cudaStream_t s);
// The step's attention launch of one layer.  `which` selects the item lists it serves (both in the
// step itself; one at a time when launches are timed per class).
constexpr int HB_ATTN_CHUNK_TILES = 1;   // chunk tiles of up to 128 rows (tcgen05 body)
constexpr int HB_ATTN_SMALL_ITEMS = 2;   // decode items (mma.sync body)
constexpr int HB_ATTN_ALL = 3;
int hb_launch_attention(hb_ctx* c, const KvGeom& kv, const CUtensorMap& kv_map, int layer, cudaStream_t s, int which);
int hb_launch_final(hb_ctx* c, const void* gain, float* pool_sum, uint32_t* pool_meta,
                    int n_slots, float* rowbuf, int rowbuf_rows, float* out_emb, cudaStream_t s);
int hb_launch_argmax(const float* logits, int n_rows, int V, int32_t* out, cudaStream_t s);
int hb_launch_wait_expiry_selftest(hb_ctx* c, uint64_t limit_ns, cudaStream_t s);
int hb_launch_pool_chunk(hb_ctx* c, const float* x, const void* gain, int n_rows, int mode, int first_chunk,
                         int is_final, float* slot_sum, uint32_t* slot_meta, float* out_emb, cudaStream_t s);
int hb_launch_bf16_to_f16(const void* src, void* dst, size_t n, cudaStream_t s);

struct hb_ctx {
  hb_model_cfg cfg;
  int32_t max_tokens, max_segs, max_page_ids;
  int num_sms;
  int device;
  bool owns_ws;
  uint8_t* ws;
  size_t ws_bytes;
  // workspace carve-up (device)
  float* x;                 // [max_tokens, d] residual stream, fp32
  __half* h;                // [max_tokens, d] normed activations (fp16)
  __half* q;                // [max_tokens, Hq*Dh] rotated queries (fp16)
  __half* attn_out;         // [max_tokens, Hq*Dh] (fp16)
  __half* act;              // [max_tokens, F] (fp16)
  __half* lora_u;           // [max_tokens, HB_LORA_U_COLS] rank-r activations of the adapted rows (fp16)
  float* lora_part;         // [HB_LORA_K_SPLITS, max_tokens, HB_LORA_U_COLS] split-K partial sums
  uint32_t* lora_counters;  // [n_lora_counters] arrival counters of the split-K merge
  int32_t n_lora_counters;
  uint32_t* resid_turns;    // [n_resid_turns] turn words of the split-K residual GEMMs (zero between launches)
  int32_t n_resid_turns;
  __half* logit_in;         // [max_logit_rows, 2d] hi/lo fp16 split of final hidden rows
  float* rope_cos;          // [max_pos, Dh/2]
  float* rope_sin;
  float* attn_part;         // split-KV partial results
  float* pool_part;         // pooling partial sums
  uint32_t* counters;       // arrival counters of the pooling merge, one per segment
  uint32_t* attn_counters;  // arrival counters of the split-KV merge, one per (segment, kv head)
  uint32_t* status;         // device status word (256-byte block: word 0 status, words 8 and 9 the attention work queue)
  uint8_t* desc_dev;        // packed descriptor
  size_t desc_cap;
  void* extra;              // host-side state (pinned descriptor staging ring, layout)
  size_t attn_part_floats, pool_part_floats;
  int32_t n_counters;
  int32_t max_logit_rows;
  DeviceDesc dd;
  // tensor maps over the activation buffers (A operands)
  CUtensorMap tm_h, tm_attn_out, tm_act, tm_logit_in, tm_lora_u;
  // cached weight tensor maps
  struct WMaps {
    const void* key[4];
    CUtensorMap qkv, o, gu, down;
    int bn_qkv, bn_o, bn_gu, bn_down;
    int ks_o, ks_down;
  };
  std::vector<WMaps> wmaps;
  // cached adapter tensor maps: down factors (B operand of the thin GEMMs), up factors (second B
  // operand of the projections)
  struct LMaps {
    const void* key[8];
    int rank;
    CUtensorMap a_qkv, b_qkv, a_o, b_o, a_gu, b_gu, a_d, b_d;
  };
  std::vector<LMaps> lmaps;
  const void* lm_key;
  CUtensorMap tm_lm;
  int32_t last_launches;
  bool pdl;   // the next launch may overlap the tail of the previous kernel (set inside a step)
};
