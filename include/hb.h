/*
 * hb.h -- C ABI of the heterogeneous-batching step library (B200 / sm_100a).
 *
 * One call, hb_mixed_step, runs ONE transformer forward over a ragged mixed
 * batch: the "forward" stage of the paper's inference loop (Algorithm 1) over
 * the batch unit of Section 3.2 (embedding chunks, generation prefill chunks,
 * decode tokens), followed by the two output paths of Algorithm 1: the
 * incremental pooler of Section 3.3 (Eq. 1-2 and the last-token head) on the
 * embedding rows and the logits for the sampler on the generation rows.
 *
 * Conventions
 *  - every function returns an int status: HB_OK (0) or a negative HB_ERR_*;
 *    nothing throws or aborts across this boundary;
 *  - "host" / "device" is stated for every pointer; device pointers are plain
 *    CUDA device addresses on the current device; `stream` is a cudaStream_t
 *    passed as void* (NULL = the legacy default stream);
 *  - the library never frees caller memory; hb_mixed_step allocates no device
 *    memory, and its host scratch (work lists, validation marks, the pinned
 *    descriptor staging) belongs to the context: it is reserved by hb_create
 *    for the context's limits and only grows if a step meets a KV cache or
 *    pool with more pages / slots than any step before (per-class timing,
 *    hb_profile_enable, creates its CUDA events on demand);
 *  - all work is enqueued on `stream`; outputs are valid once the caller has
 *    synchronised that stream;
 *  - there is no CPU path: without a CUDA device every compute call fails.
 */
#ifndef HB_H_
#define HB_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define HB_API __attribute__((visibility("default")))
#else
#define HB_API
#endif

/* ---- status codes ------------------------------------------------------- */
enum {
  HB_OK = 0,
  HB_ERR_BAD_ARG = -1,       /* null pointer, bad size, double free ...        */
  HB_ERR_CUDA = -2,          /* a CUDA runtime/driver call failed              */
  HB_ERR_OOM_PAGES = -3,     /* hb_kv_alloc_pages: not enough free pages       */
  HB_ERR_OOM_SLOTS = -4,     /* hb_pool_alloc_slot: no free slot               */
  HB_ERR_TOO_LARGE = -5,     /* batch exceeds the limits given to hb_create    */
  HB_ERR_BAD_DESC = -6,      /* batch descriptor failed validation             */
  HB_ERR_DEVICE_STATUS = -7, /* a kernel reported a bounded-wait expiry/index  */
  HB_ERR_UNSUPPORTED = -8    /* model shape outside what the kernels cover     */
};

/* Row kinds of the batch unit (Section 3.2).  Rows of one kind are contiguous
 * and kinds appear in this order (Section 3.2 has the scheduler hand over each
 * batch already grouped by kind, so every output head reads one slice). */
enum { HB_KIND_DECODE = 0, HB_KIND_PREFILL_CHUNK = 1, HB_KIND_EMBED_CHUNK = 2 };

/* Pooling heads (Section 3.3).  Additive (Eq. 1-2): mean (w = 1) and weighted
 * mean with w = 1-based position of the token in its request (the paper
 * leaves the weights open; this is the common position weighting).
 * Positional: last token (H of the last row of the final chunk) and CLS (H of
 * the first row of the first chunk, retained in the slot). */
enum { HB_POOL_NONE = 0, HB_POOL_MEAN = 1, HB_POOL_LAST = 2, HB_POOL_CLS = 3, HB_POOL_WMEAN = 4, HB_POOL_MAX = 5 };

typedef struct hb_ctx hb_ctx;
typedef struct hb_kv hb_kv;
typedef struct hb_pool hb_pool;

/* Decoder-only model: pre-norm RMSNorm, rotate-half RoPE, grouped-query causal
 * attention, SwiGLU FFN, no biases, untied LM head.  head_dim must be 64 or
 * 128; d_model, n_heads*head_dim, d_ffn multiples of 64; page_size 16.
 * Precision: bf16 model weights, repacked to fp16 for the tensor cores;
 * activations between kernels, the KV cache and the attention probabilities
 * fp16; residual stream, norms, softmax, pooling and every accumulation fp32. */
typedef struct {
  int32_t n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab;
  int32_t page_size;    /* tokens per KV page (16)                              */
  int32_t max_pos;      /* largest position + 1 any request may reach          */
  float rope_theta;
  float rms_eps;
} hb_model_cfg;

/* Weights are row-major [out, in] (y = x * W^T), device memory owned by the
 * caller.  The projection matrices are fp16: the model's bf16 values repacked
 * once with hb_weights_pack_f16 (the tensor cores take one 16-bit format for
 * both operands, and activations are fp16).  Gains and the token embedding
 * stay bf16.
 *   wqkv      fp16 [(n_heads + 2 n_kv_heads) * head_dim, d_model]: q rows, then k, then v;
 *             inside every q and k head the rows are pair-interleaved for the rotary
 *             step: row 2i = the head's row i, row 2i+1 = its row i + head_dim/2
 *             (a fixed permutation of the head dimension, applied alike to q and k,
 *             so q.k is unchanged; the KV cache holds k in this order)
 *   wo        fp16 [d_model, n_heads * head_dim]
 *   w_gate_up fp16 [2 * d_ffn, d_model]: row 2j = gate row j, row 2j+1 = up row j
 *   w_down    fp16 [d_model, d_ffn]
 *   lm_head   fp16 [vocab, d_model]
 *   attn_norm, ffn_norm, final_norm bf16 [d_model] gains
 *   tok_emb   bf16 [vocab, d_model] */
typedef struct {
  const void* attn_norm;
  const void* wqkv;
  const void* wo;
  const void* ffn_norm;
  const void* w_gate_up;
  const void* w_down;
} hb_layer_weights;

typedef struct {
  const void* tok_emb;               /* device */
  const hb_layer_weights* layers;    /* HOST array [n_layers] of device ptrs   */
  const void* final_norm;            /* device */
  const void* lm_head;               /* device */
} hb_weights;

/* One segment = the rows one request contributes to this step (Section 3.2).
 *   kind        HB_KIND_*
 *   q_start     first token row of the segment (prefix sum of q_len)
 *   q_len       rows: 1 for DECODE, chunk size c_k otherwise (>= 1)
 *   pos_start   tokens of this request already in the KV cache; row j has
 *               position pos_start + j, writes its K/V there and attends to
 *               positions 0 .. pos_start + j of its own request
 *   pt_start    offset of this request's page list inside page_ids
 *   pt_len      entries of that list; must cover pos_start + q_len tokens
 *   pool_slot   pool slot (EMBED_CHUNK) or -1
 *   pool_mode   HB_POOL_* (NONE unless EMBED_CHUNK)
 *   is_final    last chunk of the request: emit embedding / logits
 *   logits_row  row of out_logits to write (DECODE, final PREFILL_CHUNK), else -1
 *   emb_row     row of out_emb to write (final EMBED_CHUNK), else -1 */
typedef struct {
  int32_t kind, q_start, q_len, pos_start;
  int32_t pt_start, pt_len, pool_slot, pool_mode;
  int32_t is_final, logits_row, emb_row, reserved;
} hb_seg;

/* Batch descriptor; every pointer is HOST memory, read during the call only. */
typedef struct {
  int32_t n_tokens;       /* total rows T                                       */
  int32_t n_segs;         /* segments R                                         */
  int32_t n_page_ids;     /* length of page_ids                                 */
  int32_t n_logit_rows;   /* rows of out_logits produced this step              */
  int32_t n_emb_rows;     /* rows of out_emb produced this step                 */
  const int32_t* token_ids; /* [n_tokens] ids in [0, vocab)                     */
  const hb_seg* segs;       /* [n_segs]                                         */
  const int32_t* page_ids;  /* [n_page_ids] physical page numbers               */
} hb_batch_desc;

/* ---- context -------------------------------------------------------------- */

/* Bytes of device workspace a context needs for steps of at most max_tokens
 * rows, max_segs segments and max_page_ids page-list entries.  Host only. */
HB_API int hb_workspace_bytes(const hb_model_cfg* cfg, int32_t max_tokens, int32_t max_segs,
                       int32_t max_page_ids, size_t* out_bytes);

/* Create a context on the current device.  `workspace` (device, 256-byte
 * aligned, hb_workspace_bytes big) stays owned by the caller; pass NULL to let
 * the library allocate (and later free) it.  Builds the rotary table and the
 * activation tensor maps.  Synchronises the device once. */
HB_API int hb_create(const hb_model_cfg* cfg, int32_t max_tokens, int32_t max_segs,
              int32_t max_page_ids, void* workspace, size_t workspace_bytes,
              hb_ctx** out);
HB_API int hb_destroy(hb_ctx* ctx);

/* ---- paged KV cache ------------------------------------------------------- */

/* Bytes of an arena of n_pages.  Arena layout (fp16; post-rotary K and V):
 * [layer][page][kv_head][slot group][K|V][head_dim/64][8 slots][64]: slots 0-7
 * and 8-15 of a page form two groups, the head dimension is split into
 * 64-element halves, and the K+V block of one (layer, page, head) is contiguous
 * (4-8 KiB), so one TMA copy fetches it and the blocks of consecutive pages
 * line up in shared memory the way the tensor-core descriptors need.
 * Host only. */
HB_API int hb_kv_arena_bytes(const hb_model_cfg* cfg, int32_t n_pages, size_t* out_bytes);

/* Wrap a caller-owned device arena.  Only the free list lives in the library
 * (host memory); no device work.  `arena` may be NULL for host-side
 * bookkeeping tests. */
HB_API int hb_kv_create(const hb_model_cfg* cfg, void* arena, size_t arena_bytes, int32_t n_pages,
                 hb_kv** out);
HB_API int hb_kv_destroy(hb_kv* kv);
/* Take n pages (lowest free ids first); all-or-nothing: HB_ERR_OOM_PAGES. */
HB_API int hb_kv_alloc_pages(hb_kv* kv, int32_t n, int32_t* out_ids /* host [n] */);
/* Return pages; a page not currently allocated -> HB_ERR_BAD_ARG, nothing freed. */
HB_API int hb_kv_free_pages(hb_kv* kv, int32_t n, const int32_t* ids /* host [n] */);
HB_API int hb_kv_free_count(const hb_kv* kv, int32_t* out_free);

/* ---- pooling state (Section 3.3: O(d) state per request) ------------------ */

/* Arena layout: float sum[n_slots][d_model], then uint32 meta[n_slots][4] =
 * {count, chunks, mode, state}; state 0 = open, 1 = emitted.  Host only. */
HB_API int hb_pool_arena_bytes(const hb_model_cfg* cfg, int32_t n_slots, size_t* out_bytes);
HB_API int hb_pool_create(const hb_model_cfg* cfg, void* arena, size_t arena_bytes, int32_t n_slots,
                   hb_pool** out);
HB_API int hb_pool_destroy(hb_pool* pool);
/* Take a slot (lowest free id).  No device work: the first chunk of a request
 * (pos_start == 0) overwrites the slot, which realises S(0) = 0, W(0) = 0. */
HB_API int hb_pool_alloc_slot(hb_pool* pool, int32_t* out_slot);
HB_API int hb_pool_free_slot(hb_pool* pool, int32_t slot);

/* Row buffer for buffered heads (Section 3.3: a head that is neither additive
 * nor positional keeps A(k) = [A(k-1); H(k)], every final hidden state of the
 * request, at O(n d) memory, and runs after the final chunk).  Layout:
 * float rows[n_slots][max_rows][d_model]; row p of a slot holds the final
 * RMSNorm output of the request's token at position p.  The caller owns the
 * memory (device, 256-byte aligned); attach it once, before the first step
 * that uses HB_POOL_MAX.  HB_POOL_MAX is the buffered head built in: every
 * chunk appends its rows, the final chunk emits the element-wise maximum over
 * all n rows, L2-normalised.  After the final chunk the buffer holds all n
 * rows, so a caller can run any other head over them itself.  A segment with
 * pos_start + q_len > max_rows, or HB_POOL_MAX without an attached buffer, is
 * HB_ERR_BAD_DESC.  max_rows in 1..cfg.max_pos.  Host only. */
HB_API int hb_pool_row_buffer_bytes(const hb_model_cfg* cfg, int32_t n_slots, int32_t max_rows, size_t* out_bytes);
HB_API int hb_pool_attach_row_buffer(hb_pool* pool, void* buf, size_t bytes, int32_t max_rows);

/* ---- the step ------------------------------------------------------------- */

/* Host-only validation of a descriptor against the limits (what hb_mixed_step
 * checks before it enqueues anything): sizes, kind order, q_start prefix sums,
 * page lists cover pos_start + q_len, page ids in [0, n_pages), a page written
 * this step belongs to one segment only, pool slots in range and used once,
 * output rows in range and used once, token ids in range. */
HB_API int hb_validate_desc(const hb_model_cfg* cfg, int32_t max_tokens, int32_t max_segs,
                     int32_t max_page_ids, int32_t n_pages, int32_t n_slots,
                     const hb_batch_desc* desc);

/* One forward step over the mixed batch (Algorithm 1: Forward, IncPooler,
 * and the logits the Sampler consumes).
 *   desc        host descriptor (copied; may be reused after return)
 *   w           host struct of device weight pointers
 *   kv, pool    caches created above; K/V of every row is appended to its
 *               page; pool slots of EMBED_CHUNK segments are updated
 *   out_logits  device float [>= n_logit_rows, vocab]; row seg.logits_row gets
 *               the logits of the segment's last row
 *   out_emb     device float [>= n_emb_rows, d_model]; row seg.emb_row gets the
 *               L2-normalised embedding of a request whose final chunk ran
 * Rows of the outputs not named by a segment are left untouched.  Returns
 * after enqueueing; no synchronisation, no device allocation.  A failed
 * validation enqueues nothing.  Alignment (checked, HB_ERR_BAD_ARG): out_logits,
 * out_emb and tok_emb 16 bytes, every norm gain 8 bytes (the kernels use
 * 16-byte and 8-byte vector accesses); projection weights 16 bytes. */
HB_API int hb_mixed_step(hb_ctx* ctx, const hb_batch_desc* desc, const hb_weights* w, hb_kv* kv,
                  hb_pool* pool, float* out_logits, float* out_emb, void* stream);

/* ---- low-rank adapters on embedding rows ------------------------------------
 *
 * With a shared backbone the embedding model is the generation model plus a
 * low-rank adapter (Section 2.1, paragraph on parameter sharing; in Section
 * 5.1 both request types share one GPU through such adapters).  Inside the one forward
 * pass, rows of EMBED_CHUNK segments compute every projection as
 *     y = x W^T + (alpha / r) (x A^T) B^T,        A [r, in], B [out, r],
 * and rows of DECODE / PREFILL_CHUNK segments compute y = x W^T.  The paper
 * does not say which projections carry the adapter; here all seven of a layer
 * do (q, k, v, o, gate, up, down).  Token embedding, norm gains and LM head
 * are shared unchanged.
 *
 * Packed layout (device, fp16, row-major, 16-byte aligned; the caller packs
 * once).  R(n) = n * r rounded up to a multiple of 64; unused rows / columns
 * are zero.  Row orders of the B factors follow the fused weights they pair
 * with (hb_layer_weights):
 *   a_qkv  [R(3), d]          rows [0,r) = A_q, [r,2r) = A_k, [2r,3r) = A_v
 *   b_qkv  [(Hq+2Hkv)Dh, R(3)] rows as wqkv (q and k rows pair-interleaved per
 *                             head); q rows hold B_q in columns [0,r), k rows
 *                             B_k in [r,2r), v rows B_v in [2r,3r), zero elsewhere
 *   a_o    [R(1), Hq*Dh]      A_o;           b_o  [d, R(1)]   B_o
 *   a_gu   [R(2), d]          A_gate, A_up;  b_gu [2F, R(2)]  rows as w_gate_up
 *                             (gate_j, up_j interleaved): gate rows hold B_gate
 *                             in [0,r), up rows B_up in [r,2r)
 *   a_d    [R(1), F]          A_down;        b_d  [d, R(1)]   B_down
 * scale = alpha / r multiplies the rank-r activations in fp32 before they are
 * rounded to fp16.  rank in 1..64. */
typedef struct hb_lora_layer {
  const void *a_qkv, *b_qkv, *a_o, *b_o, *a_gu, *b_gu, *a_d, *b_d;
} hb_lora_layer;

typedef struct hb_lora {
  int32_t rank;
  float scale;
  const hb_lora_layer* layers; /* host array [n_layers] */
} hb_lora;

/* hb_mixed_step with adapters on the EMBED_CHUNK rows.  lora == NULL, or a
 * step without EMBED_CHUNK rows, is exactly hb_mixed_step.  Per layer this
 * adds four thin GEMMs (the rank-r activations of the rows, zero for rows
 * that carry no adapter) and extends the K loop of the four projection GEMMs
 * by R / 64 blocks.  The context must have been created after
 * hb_workspace_bytes (the workspace always includes the rank-r buffer). */
HB_API int hb_mixed_step_lora(hb_ctx* ctx, const hb_batch_desc* desc, const hb_weights* w, const hb_lora* lora,
                       hb_kv* kv, hb_pool* pool, float* out_logits, float* out_emb, void* stream);

/* Repack bf16 values to fp16, element by element, on `stream` (device
 * pointers, 16-byte aligned; dst may equal src for an in-place repack, partial
 * overlap is rejected).  Exact for 2^-14 <= |w| <= 65504; smaller magnitudes
 * round to the fp16 subnormal grid (absolute error <= 2^-25), larger saturate. */
HB_API int hb_weights_pack_f16(const void* src_bf16, void* dst_f16, size_t n_elems, void* stream);

/* Greedy sampler over logits rows (Algorithm 1 "Sampler", greedy case): lowest
 * index of the maximum of each row.  logits device float [n_rows, vocab],
 * out_tokens device int32 [n_rows]. */
HB_API int hb_argmax(hb_ctx* ctx, const float* logits, int32_t n_rows, int32_t* out_tokens,
              void* stream);

/* Read (and clear) the device status word; synchronises `stream`.  0 = clean.
 * Non-zero: *out_code holds the OR of the bits below and the call returns
 * HB_ERR_DEVICE_STATUS.  Bits 0-5 mean a kernel gave up (a bounded wait expired,
 * an index check failed: outputs of that step are not valid); bit 6 is a value
 * report: the step ran, but an activation did not fit fp16. */
enum {
  HB_STATUS_GEMM_WAIT = 1,        /* projection GEMM: a pipeline wait expired                 */
  HB_STATUS_ATTN_INDEX = 2,       /* attention: page id out of range                          */
  HB_STATUS_APPEND_INDEX = 4,     /* KV append: page id out of range (row not written)        */
  HB_STATUS_POOL_INDEX = 8,       /* pooler: slot / row buffer out of range                   */
  HB_STATUS_ATTN_WAIT = 16,       /* attention: a pipeline wait expired                       */
  HB_STATUS_SELFTEST_WAIT = 32,   /* hb_selftest_wait_expiry                                  */
  HB_STATUS_F16_RANGE = 64        /* a normed row or a SwiGLU output was NaN or beyond +-65504:
                                     finite values were stored saturated, NaN was stored as NaN */
};
HB_API int hb_status_poll(hb_ctx* ctx, void* stream, uint32_t* out_code);

/* Per-kernel-class device timing.  While enabled, hb_mixed_step brackets every launch with a
 * pair of CUDA events on the step's stream; hb_profile_read synchronises them, adds the
 * elapsed milliseconds and launch counts per class into the two arrays of HB_N_CLASSES
 * entries, and clears the record.  While enabled, launches do not overlap one another and
 * the layer's one attention launch is issued once per item list (classes 1 and 5), so the
 * launch count of a step is higher than in normal operation.  Classes: */
enum {
  HB_CLASS_GEMM = 0,      /* QKV, O, gate/up, down projections                          */
  HB_CLASS_ATTENTION = 1, /* attention launch (when timed: the decode splits alone) */
  HB_CLASS_NORM_ROPE = 2, /* gather + RMSNorm, RMSNorm, RoPE + KV append                */
  HB_CLASS_POOL = 3,      /* final RMSNorm + pooler / logits-row preparation            */
  HB_CLASS_LM_HEAD = 4,   /* LM-head projection                                         */
  HB_CLASS_ATTENTION_TC = 5, /* when timed: the attention launch's tcgen05 chunk tiles alone */
  HB_CLASS_LORA = 6,      /* adapters: rank-r activations of the embedding rows         */
  HB_N_CLASSES = 7
};
HB_API int hb_profile_enable(hb_ctx* ctx, int on);
HB_API int hb_profile_read(hb_ctx* ctx, float* ms_by_class, int32_t* launches_by_class);

/* Failure-path self-test.  Every wait inside the kernels (on an mbarrier fed by TMA, by the tensor
 * cores or by another warp role) is bounded in time; when a bound expires the kernel raises a bit
 * in the status word and returns normally.  This call launches a one-thread kernel that runs the
 * same bounded wait on a barrier nothing arrives on, with a limit of limit_ms (1..1000)
 * milliseconds, so that the path "wait expires -> status bit -> hb_status_poll returns
 * HB_ERR_DEVICE_STATUS -> context still usable" can be exercised without faulting or hanging the
 * GPU.  The status code it raises is 32. */
HB_API int hb_selftest_wait_expiry(hb_ctx* ctx, uint32_t limit_ms, void* stream);

/* Kernels launched by the last hb_mixed_step on this context. */
HB_API int hb_last_launch_count(const hb_ctx* ctx, int32_t* out_count);

/* ---- kernel-level entry points (used by the parity tests) ----------------- */

/* Epilogues of the projection GEMM (the dense contractions of the forward,
 * Section 3.1: the attention and feed-forward projections every row passes through). */
enum {
  HB_EPI_F16 = 0,       /* C fp16 [M,N] = A * B^T                               */
  HB_EPI_F32 = 1,       /* C float [M,N] = A * B^T                              */
  HB_EPI_RESID_F32 = 2, /* C float [M,N] += A * B^T (residual stream update)    */
  HB_EPI_SWIGLU = 3     /* C fp16 [M,N/2]: silu(acc[2j]) * acc[2j+1]            */
};

/* C = epilogue(A * B^T): A fp16 [M,K] row-major (activations), B fp16 [N,K]
 * row-major (weights), both K-major, fp32 accumulation on the tcgen05 tensor
 * cores; fp16 outputs saturate at +-65504.  All device pointers, 16-byte
 * aligned; K and N multiples of 8.  M may be any value >= 1. */
HB_API int hb_gemm(hb_ctx* ctx, const void* A, const void* B, void* C, int32_t M, int32_t N,
            int32_t K, int32_t epilogue, void* stream);

/* hb_gemm with a second operand pair accumulated after the first:
 * C = epilogue(A * B^T + A2 * B2^T), A2 fp16 [M,K2], B2 fp16 [N,K2], K2 a
 * multiple of 64.  This is how an adapted projection adds its low-rank branch
 * (hb_mixed_step_lora): A2 = the rows' rank-r activations, B2 = the up factor. */
HB_API int hb_gemm_pair(hb_ctx* ctx, const void* A, const void* B, const void* A2, const void* B2, void* C,
                 int32_t M, int32_t N, int32_t K, int32_t K2, int32_t epilogue, void* stream);

/* Tile walk of the projection GEMM, for tests and tuning.  A launch normally chooses by itself in
 * which order its workers take the output tiles (rows fastest over the whole M, or in bands of row
 * tiles when A's share of a work item would not stay in L2) and whether its loads carry L2 eviction
 * hints.  The walk never changes the K order of an element's sum, so results are bit-identical under
 * every setting; this call forces one for all later launches of the process so that a test can show
 * exactly that, and a profile can compare DRAM traffic.  band >= 1: row tiles per band; band = 0: whole
 * M; hints 0 / 1; -1 for either = automatic again.  Host only, not thread-safe against launches. */
HB_API int hb_gemm_set_walk(int32_t band, int32_t hints);
/* Tuning: cap the CTAs of every projection launch at max_ctas (even; 0 = one per SM again), e.g. to
 * leave SMs to kernels of another stream.  Changes the work split between workers only, never a
 * result bit.  Host only, process-wide. */
HB_API int hb_gemm_set_cta_limit(int32_t max_ctas);
/* The attention launch of a step runs min(items, 2 per SM) resident blocks that take the step's
 * attention items (decode splits, chunk tiles) one after the other from a ticket.  This call caps the
 * blocks of every later attention launch of the process at max_blocks (0 = automatic again), so that a
 * test can make one block walk through many items of both kinds.  Which block runs an item never
 * changes a result bit (an item's arithmetic is its own; the splits of a decode row are merged in
 * split order by whichever block arrives last).  Host only, not thread-safe against launches. */
HB_API int hb_attn_set_block_limit(int32_t max_blocks);
/* Keys per decode attention item.  A decode row with n = context + 1 keys is cut into
 * max(1, (n + keys / 2) div keys) equal splits (rounded up to whole 64-key tiles) that different blocks
 * may run; their partial results are merged in split order.  The count depends on the row's own context
 * and on this value only, never on the rest of the batch, so a request's result does not depend on its
 * batch; it does depend on this value (another summation order: results differ in the last bits).
 * Default 2048 (keys = 0 restores it); multiples of 64 from 256 to 65536.  A smaller value keeps more
 * blocks busy when steps hold only a few long decode rows, at the cost of a partial record, a fence, an
 * atomic and a share of the merge per split.  Process-wide; hb_workspace_bytes and hb_create read it,
 * and a context keeps the value it was created with.  Host only. */
HB_API int hb_attn_set_split_keys(int32_t keys);

/* The incremental pooler on its own (Section 3.3, Eq. 1-2 and the last-token
 * head), as hb_mixed_step runs it on an embedding segment: final RMSNorm of
 * the chunk's rows, then
 *   mean / weighted mean: S <- S + sum_j w_j rmsnorm(x_j) * gain, count <-
 *         count + n_rows (first_chunk != 0 starts from S = 0, count = 0; the
 *         position weights continue from the slot's count);
 *   last: only the counters move until the final chunk; cls: the first
 *         chunk's first normed row is kept in S;
 * and on the final chunk out_emb = L2-normalised S / W (W = count, or
 * count (count + 1) / 2 for position weights) or the retained row.
 *   x          device float [n_rows, d_model] residual-stream rows of the chunk
 *   gain       device bf16 [d_model] final-norm gain
 *   slot_sum   device float [d_model], slot_meta device uint32 [4] =
 *              {count, chunks, mode, state}: the request's pool slot (in/out)
 *   out_emb    device float [d_model] (written when is_final != 0)
 * n_rows <= the context's max_tokens.  Uses the context's scratch.  x,
 * slot_sum and out_emb must be 16-byte aligned, gain 8-byte aligned (vector
 * accesses); a misaligned pointer is HB_ERR_BAD_ARG and nothing is launched. */
HB_API int hb_pool_chunk(hb_ctx* ctx, const float* x, const void* gain, int32_t n_rows, int32_t mode,
                         int32_t first_chunk, int32_t is_final, float* slot_sum, uint32_t* slot_meta,
                         float* out_emb, void* stream);

/* ---- entry point that allocates nothing ------------------------------------ */

/* Largest chunk and hidden size hb_pool_chunk_noalloc accepts. */
#define HB_NOALLOC_MAX_ROWS 2048
#define HB_NOALLOC_MAX_DMODEL 4096

/* (The paper has no counterpart to this call; it exists for deployment.)
 * hb_pool_chunk without a context and without any allocation: same arguments
 * and results as hb_pool_chunk, with d_model and rms_eps passed directly.
 *
 * Who needs it: a caller that cannot allocate device memory -- for example a
 * serving process whose own allocator claimed the whole device at start-up, or
 * code running where a device allocation would fail or stall the GPU -- cannot
 * create an hb_ctx (that allocates the workspace) and so cannot reach any other
 * compute call.  Here the pooler's scratch (partial sums of 32-row blocks, an
 * arrival counter, a status word) lives in a fixed array inside the library
 * image instead: 1 MiB + 256 bytes on every GPU that loads the library, held
 * until the process exits.  The call itself uses no cudaMalloc, cudaFree or
 * any other allocating routine.
 *
 * Limits and rules
 *  - n_rows <= HB_NOALLOC_MAX_ROWS and d_model <= HB_NOALLOC_MAX_DMODEL
 *    (d_model a multiple of 4); anything larger returns HB_ERR_TOO_LARGE and
 *    does nothing;
 *  - the first call on a device looks up the array's device address (once per
 *    device, with that device current); make that first call before starting
 *    any stream capture;
 *  - all calls on a device share the one array, which keeps the previous
 *    call's contents (the call clears the words that must start at zero).
 *    Two calls whose kernels can run at the same time on that device -- from
 *    different streams or threads -- race on it: serialise them;
 *  - the caller still owns and passes every input and output (x, gain,
 *    slot_sum, slot_meta, out_emb: device pointers as in hb_pool_chunk), with
 *    the same alignment rule: x, slot_sum, out_emb 16 bytes, gain 8 bytes.  A
 *    view cut out of a larger arena at an odd offset is refused with
 *    HB_ERR_BAD_ARG before anything is launched;
 *  - the looked-up address is cached for the life of the process.  After
 *    cudaDeviceReset on that device it is stale: do not call this entry again
 *    in a process that reset the device;
 *  - there is no context, so no hb_status_poll: the status word the kernel
 *    keeps in the array's tail is write-only for callers.  The only device
 *    check behind it (pool slot in range) cannot fail here, because this entry
 *    always runs on a one-slot pool it builds itself. */
HB_API int hb_pool_chunk_noalloc(const float* x, const void* gain, int32_t n_rows, int32_t d_model,
                                 float rms_eps, int32_t mode, int32_t first_chunk, int32_t is_final,
                                 float* slot_sum, uint32_t* slot_meta, float* out_emb, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* HB_H_ */
