// Attention over the paged KV cache for decode rows (Section 3.2 of the paper: decode tokens attend
// over their cached context).  A decode row at position pos sees keys 0 .. pos of its own request; all
// keys, the row's own included, are read from the pages (the projection's epilogue appended them
// before).  Chunk rows take the tcgen05 body (attention_tc.cuh), whatever the size of their tile: a
// 64-row remainder costs that body less per key tile than it cost this one.
//
// Work items come from the batch descriptor (host-built list):
//   decode item  the G query heads of one KV head (G = Hq / Hkv) of one decode row over one split of
//                its keys; the four warps share the rows and own 16 keys of every 64-key tile;
//                their partial (max, sum, output) are merged in shared memory, and the splits
//                of a row through a scratch record per split, merged in split order by the CTA
//                that arrives last (integer arrival counter; no floating-point atomics).
// K/V tiles of 64 keys (4 pages) are gathered by TMA: one 2-D tensor copy per page (the contiguous
// K+V block of this KV head, 4-8 KiB: the TMA unit's rate is per copy, so few large copies) into a
// 128-byte-swizzled shared-memory ring; the CTA waits on the stage's mbarrier (bounded).
// S = Q K^T and O += P V run on mma.sync m16n8k16 (fp16 in, fp32 accumulate), softmax in fp32 with
// exp2.  Split decisions depend on the request's own length only, so a request's result does not
// depend on its batch mates.
//
// This file is the body of one CTA; attention.cu includes it and calls it from the one attention
// kernel of the step for the blocks that hold such an item.
#pragma once
#include "hb_internal.h"
#include "ptx.cuh"

namespace hb_dec {

// Four compute warps, one warp that drives TMA, and one warp that only keeps the block barriers
// company: the kernel's block size is the one the tensor-core chunk items need.
constexpr int ATT_THREADS = 192;
constexpr int ATT_COMPUTE = 128;
constexpr int TILE_KEYS = 64;
constexpr int TILE_ROWS = 64;
constexpr int STAGES = 3;
constexpr uint64_t ATT_WAIT_NS = 1000000000ull;  // 1 s

struct AttnParams {
  const __half* q;            // [T, Hq*Dh] fp16
  __half* out;                // [T, Hq*Dh] fp16
  KvGeom kv;
  int layer;
  const AttnItem* items;
  const int32_t* pages;
  float* part;                // split records: [record][G][Dh + 2]
  uint32_t* counters;         // [seg * Hkv + kv_head]
  uint32_t* status;
  int Hq, G;
  float scale_log2;           // log2(e) / sqrt(Dh)
};

// Byte offset of 16-byte chunk `c` of row `r` in a 64-row tile stored as [DH/64 halves][64 rows][64]
// bf16 with the 128-byte swizzle TMA applies (chunk index XOR row mod 8 inside each 128-byte row).
template <int DH>
__device__ __forceinline__ uint32_t tile_off(int r, int c) {
  return static_cast<uint32_t>((c >> 3) * (64 * 128) + r * 128 + (((c & 7) ^ (r & 7)) << 4));
}

// Byte offset of 16-byte chunk `c` of key `r` of a 64-key K/V tile as TMA lands it: four page blocks
// of DH*64 bytes, each [slot group][K|V][DH/64 halves][8 keys][64] (the arena's own layout), 128-byte
// swizzle inside every row.
template <int DH>
__device__ __forceinline__ uint32_t kv_off(int r, int c, int is_v) {
  return static_cast<uint32_t>((r >> 4) * (DH * 64) + ((r >> 3) & 1) * (DH * 32) + (is_v * (DH / 64) + (c >> 3)) * 1024 +
                               (r & 7) * 128 + (((c & 7) ^ (r & 7)) << 4));
}

// One warp: 16 query rows against NT*8 keys starting at tile-local key `kofs`.
// qf: Q fragments; m, l: running max (scaled, log2 domain) and per-thread partial sums of the two
// rows this thread touches (row lane/4 and row lane/4 + 8); oacc: unnormalised output.
template <int DH, int NT>
__device__ __forceinline__ void warp_attend(const uint32_t (&qf)[DH / 16][4], uint32_t kv_tile,
                                            int kofs, int key_base, int key_end, int pos_a, int pos_b,
                                            float scale_log2, float (&m)[2], float (&l)[2],
                                            float (&oacc)[DH / 8][4]) {
  const int lane = threadIdx.x & 31;
  float s[NT][4];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.0f;
  // S = Q K^T
  {
    const int j = lane >> 3, rr = lane & 7;
#pragma unroll
    for (int ks = 0; ks < DH / 16; ++ks) {
#pragma unroll
      for (int np = 0; np < NT / 2; ++np) {
        const int key = kofs + np * 16 + (j >> 1) * 8 + rr;
        uint32_t b[4];
        ldsm_x4(kv_tile + kv_off<DH>(key, ks * 2 + (j & 1), 0), b);
        mma_f16(s[np * 2], qf[ks], b[0], b[1]);
        mma_f16(s[np * 2 + 1], qf[ks], b[2], b[3]);
      }
    }
  }
  // mask + online softmax
  float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int key = key_base + kofs + nt * 8 + 2 * (lane & 3) + (e & 1);
      const int pos = (e < 2) ? pos_a : pos_b;
      const bool vis = (key <= pos) && (key < key_end);
      s[nt][e] = vis ? s[nt][e] * scale_log2 : -INFINITY;
      mx[e >> 1] = fmaxf(mx[e >> 1], s[nt][e]);
    }
  }
  float corr[2], msafe[2];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
    mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
    const float m_new = fmaxf(m[h], mx[h]);
    msafe[h] = (m_new == -INFINITY) ? 0.0f : m_new;
    corr[h] = exp2f(m[h] - msafe[h]);   // m = -inf -> 0
    m[h] = m_new;
  }
  float rs[2] = {0.0f, 0.0f};
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float p = exp2f(s[nt][e] - msafe[e >> 1]);
      s[nt][e] = p;
      rs[e >> 1] += p;
    }
  }
  l[0] = l[0] * corr[0] + rs[0];
  l[1] = l[1] * corr[1] + rs[1];
#pragma unroll
  for (int dn = 0; dn < DH / 8; ++dn) {
    oacc[dn][0] *= corr[0]; oacc[dn][1] *= corr[0];
    oacc[dn][2] *= corr[1]; oacc[dn][3] *= corr[1];
  }
  // O += P V
  {
    const int j = lane >> 3, rr = lane & 7;
#pragma unroll
    for (int kp = 0; kp < NT / 2; ++kp) {
      uint32_t a[4];
      a[0] = pack_half2(s[kp * 2][0], s[kp * 2][1]);
      a[1] = pack_half2(s[kp * 2][2], s[kp * 2][3]);
      a[2] = pack_half2(s[kp * 2 + 1][0], s[kp * 2 + 1][1]);
      a[3] = pack_half2(s[kp * 2 + 1][2], s[kp * 2 + 1][3]);
      const int key = kofs + kp * 16 + (j & 1) * 8 + rr;
#pragma unroll
      for (int dp = 0; dp < DH / 16; ++dp) {
        uint32_t b[4];
        ldsm_x4_trans(kv_tile + kv_off<DH>(key, dp * 2 + (j >> 1), 1), b);
        mma_f16(oacc[dp * 2], a, b[0], b[1]);
        mma_f16(oacc[dp * 2 + 1], a, b[2], b[3]);
      }
    }
  }
}

// Dynamic shared memory one item needs: ring + barriers + page ids of one item (at most every page
// of a request) + alignment slack.
template <int DH>
constexpr int smem_bytes(int max_pos) { return TILE_KEYS * DH * 2 * (2 * STAGES) + 64 + (max_pos / 16 + 2) * 4 + 1024; }

// The item's barrier words stop being barriers (the block's next item may lay its shared memory out
// differently).  One thread, after the block has met at a barrier.
template <int DH>
__device__ __forceinline__ void retire_barriers(uint32_t smem_base) {
  const uint32_t kv_s = (smem_base + 1023u) & ~1023u;
  for (int st = 0; st < STAGES; ++st) mbar_inval(kv_s + STAGES * 2 * (TILE_KEYS * DH * 2) + 8u * st);
}

// One CTA of ATT_THREADS threads, item `item` of p.items.  `kv_map_p` points at the kernel's
// __grid_constant__ tensor map.  Returns false in thread 0 when the block must not take further items.
// `at_start` is called once, first thing, by thread ATT_COMPUTE + 32 (first lane of the warp that
// neither computes nor talks to TMA): whatever it waits for hides behind the item's first loads.
template <int DH, class AtStart>
__device__ __forceinline__ bool small_item(const CUtensorMap* kv_map_p, const AttnParams& p, int item, AtStart&& at_start) {
  constexpr int CH = DH / 8;                          // 16-byte chunks per row
  constexpr int TILE_BYTES = TILE_KEYS * DH * 2;
  constexpr int REC = DH + 2;                         // floats per row of a partial record
  extern __shared__ uint8_t smem_raw[];
  // carve-up (1024-byte aligned for the TMA swizzle): STAGES x (K tile, V tile) | barriers, flag | page ids.
  // The Q tile borrows the K half of the last stage until the fragments are in registers.
  const uint32_t kv_s = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (kv_s - smem_u32(smem_raw));
  const uint32_t q_s = kv_s + (STAGES - 1) * 2 * TILE_BYTES;
  const uint32_t bar_s = kv_s + STAGES * 2 * TILE_BYTES;
  uint32_t& is_last_s = *reinterpret_cast<uint32_t*>(smem + STAGES * 2 * TILE_BYTES + 32);
  int32_t* pg_s = reinterpret_cast<int32_t*>(smem + STAGES * 2 * TILE_BYTES + 64);

  const AttnItem it = p.items[item];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = p.G, Hq = p.Hq;
  if (it.mode == 0) {   // chunk tiles all go to the tcgen05 body; the host never lists one here
    if (tid == 0) atomicOr(p.status, HB_DEV_ATTN_BAD_INDEX);
    return false;
  }
  const int hk = it.kv_head;

  const int n_tiles = (it.key1 - it.key0 + TILE_KEYS - 1) / TILE_KEYS;
  const int first_blk = it.key0 / p.kv.P;
  const int n_blk = (it.key1 + p.kv.P - 1) / p.kv.P - first_blk;
  constexpr int PAGE_BYTES = DH * 64;
  // one thread: request the pages of tile kt from TMA, one copy (K and V of this head) per page
  auto issue_pages = [&](int kt, const int (&ids)[TILE_KEYS / 16]) {
    const int st = kt % STAGES;
    const uint32_t k_dst = kv_s + st * 2 * TILE_BYTES, bar = bar_s + 8u * st;
    const int kb = it.key0 + kt * TILE_KEYS;
    const int n_pg = min(TILE_KEYS / 16, (it.key1 - kb + 15) / 16);
    mbar_arrive_expect_tx(bar, static_cast<uint32_t>(n_pg) * PAGE_BYTES);
#pragma unroll
    for (int pi = 0; pi < TILE_KEYS / 16; ++pi) {
      if (pi < n_pg) {
        const int row = static_cast<int>(((static_cast<int64_t>(p.layer) * p.kv.n_pages + ids[pi]) * p.kv.Hkv + hk) * (DH / 2));
        tma_load_2d(k_dst + pi * PAGE_BYTES, kv_map_p, bar, 0, row);
      }
    }
  };
  auto issue_tile = [&](int kt) {
    int ids[TILE_KEYS / 16];
    const int pi0 = (it.key0 + kt * TILE_KEYS) / 16 - first_blk;
#pragma unroll
    for (int pi = 0; pi < TILE_KEYS / 16; ++pi) ids[pi] = (pi0 + pi < n_blk) ? pg_s[pi0 + pi] : 0;
    issue_pages(kt, ids);
  };
  // The thread that talks to TMA sits in a warp of its own: requesting a tile (page ids, four copies,
  // the proxy fence) takes ~650 cycles, which on a compute warp made that warp the one every block
  // barrier waited for.
  const bool prod = (tid == ATT_COMPUTE);
  const bool compute = (warp < ATT_COMPUTE / 32);
  int issued = 0, bad = 0;
  if (warp == ATT_COMPUTE / 32) {
    if (lane == 0) {
      for (int st = 0; st < STAGES; ++st) mbar_init(bar_s + 8u * st, 1);
      mbar_init_fence();
    }
    __syncwarp();
    // The first tiles are requested right away, with page ids read straight from global memory, so
    // that their latency overlaps the rest of the set-up; one lane per page (a single thread needs
    // ~650 cycles per tile, which for a short item is most of its start-up).
    static_assert((STAGES - 1) * (TILE_KEYS / 16) <= 32, "one lane per page of the first tiles");
    const int n_init = min(STAGES - 1, n_tiles);
    const int t0 = lane / (TILE_KEYS / 16), pi = lane % (TILE_KEYS / 16);
    const bool act = (t0 < n_init) && (lane < n_blk);
    int id = 0;
    if (act) {
      const int blk = first_blk + lane;
      id = (blk < it.pt_len) ? __ldg(p.pages + it.pt_start + blk) : -1;
      bad = (id < 0 || id >= p.kv.n_pages);
    }
    bad = __any_sync(0xffffffffu, bad);
    if (!bad) {
      const uint32_t bar = bar_s + 8u * t0;
      if (t0 < n_init && pi == 0) {
        const int n_pg = min(TILE_KEYS / 16, (it.key1 - (it.key0 + t0 * TILE_KEYS) + 15) / 16);
        mbar_arrive_expect_tx(bar, static_cast<uint32_t>(n_pg) * PAGE_BYTES);
      }
      __syncwarp();
      if (act) {
        const int row = static_cast<int>(((static_cast<int64_t>(p.layer) * p.kv.n_pages + id) * p.kv.Hkv + hk) * (DH / 2));
        tma_load_2d(kv_s + t0 * 2 * TILE_BYTES + pi * PAGE_BYTES, kv_map_p, bar, 0, row);
      }
      issued = n_init;
    }
  }
  if (tid == ATT_COMPUTE + 32) at_start();
  // page ids of the keys this item reads -> shared memory (checked once)
  for (int i = tid; i < n_blk; i += ATT_THREADS) {
    const int blk = first_blk + i;
    const int pg = (blk < it.pt_len) ? p.pages[it.pt_start + blk] : -1;
    bad |= (pg < 0 || pg >= p.kv.n_pages);
    pg_s[i] = pg;
  }
  // ---- Q rows -> shared memory: the 16 rows of the one MMA row tile (rows past n_rows are zero) ----
  for (int u = tid; u < 16 * CH; u += ATT_THREADS) {
    const int rr = u / CH, c = u - rr * CH;
    const int r = it.row0 + rr;
    const bool valid = rr < it.n_rows;
    const int tok = it.q_start + (valid ? r / G : 0), head = hk * G + (valid ? r % G : 0);
    const __half* src = p.q + (static_cast<size_t>(tok) * Hq + head) * DH + c * 8;
    cp_async16(q_s + tile_off<DH>(rr, c), src, valid);
  }
  cp_async_commit();
  if (__syncthreads_or(bad)) {  // also publishes the barrier initialisation and the page ids
    if (prod) {
      atomicOr(p.status, HB_DEV_ATTN_BAD_INDEX);
      for (int st = 0; st < issued; ++st) mbar_wait(bar_s + 8u * st, 0u, nullptr, ATT_WAIT_NS);   // copies already requested must land
    }
    cp_async_wait<0>();
    __syncthreads();
    return false;
  }

  // rows of this thread: rows 0..15 of the tile for every warp (the G heads of the decode row first)
  constexpr int row_base = 0;
  const int ra = row_base + (lane >> 2), rb = ra + 8;
  // position of the rows (rows past n_rows get -1: nothing visible)
  const int pos_a = (ra < it.n_rows) ? it.pos_start + (it.row0 + ra) / G : -1;
  const int pos_b = (rb < it.n_rows) ? it.pos_start + (it.row0 + rb) / G : -1;

  uint32_t qf[DH / 16][4];
  float m[2] = {-INFINITY, -INFINITY}, l[2] = {0.0f, 0.0f};
  float oacc[DH / 8][4];
#pragma unroll
  for (int dn = 0; dn < DH / 8; ++dn) oacc[dn][0] = oacc[dn][1] = oacc[dn][2] = oacc[dn][3] = 0.0f;

  // A wait that expires is remembered; control flow stays uniform (every thread keeps meeting the
  // block barriers) and the CTA leaves at the next loop head without storing anything.
  int failed = 0;
  cp_async_wait<0>();
  for (int kt = 0; kt < n_tiles; ++kt) {
    if (__syncthreads_or(failed)) { failed = 1; break; }   // everyone is done with tile kt - 1 (and Q landed)
    if (prod && kt > 0) {   // at kt = 0 the last stage still holds Q
      fence_async_smem();  // stages were read / patched by generic accesses
      for (; issued < n_tiles && issued < kt + STAGES; ++issued) issue_tile(issued);
    }
    if (kt == 0 && compute) {
      const int j = lane >> 3, rr = lane & 7;
#pragma unroll
      for (int ks = 0; ks < DH / 16; ++ks)
        ldsm_x4(q_s + tile_off<DH>(row_base + (j & 1) * 8 + rr, ks * 2 + (j >> 1)), qf[ks]);
    }
    const uint32_t k_tile = kv_s + (kt % STAGES) * 2 * TILE_BYTES;
    const int key_base = it.key0 + kt * TILE_KEYS;
    if (compute &&
        !mbar_wait(bar_s + 8u * (kt % STAGES), static_cast<uint32_t>((kt / STAGES) & 1), nullptr, ATT_WAIT_NS))
      failed = 1;
    const int valid_rows = it.key1 - key_base;
    if (valid_rows < TILE_KEYS) {
      // rows past the last key hold stale bytes (rest of the last page, pages not requested): zero the
      // V rows so that a zero probability times garbage cannot produce NaN (K rows are masked anyway)
      uint8_t* kv_gen = smem + (kt % STAGES) * 2 * TILE_BYTES;
      // (compute warps only: they have seen the tile land; the TMA warp has not waited for it)
      for (int u = tid; compute && u < (TILE_KEYS - valid_rows) * CH; u += ATT_COMPUTE) {
        const int rr = valid_rows + u / CH, c = u % CH;
        *reinterpret_cast<uint4*>(kv_gen + kv_off<DH>(rr, c, 1)) = make_uint4(0u, 0u, 0u, 0u);
      }
      __syncthreads();
    }
    // (the TMA warp and the sixth warp have nothing to compute)
    if (compute && key_base + warp * 16 < it.key1)
      warp_attend<DH, 2>(qf, k_tile, warp * 16, key_base, it.key1, pos_a, pos_b, p.scale_log2, m, l, oacc);
  }
  if (__syncthreads_or(failed)) {
    if (prod) {
      atomicOr(p.status, HB_DEV_ATTN_WAIT_EXPIRED);
      for (int i = 0; i < 200; ++i) __nanosleep(1000);  // let requested copies land before the block goes on
    }
    __syncthreads();
    return false;
  }
  // row sums: add the four threads of a quad
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    l[h] += __shfl_xor_sync(0xffffffffu, l[h], 1);
    l[h] += __shfl_xor_sync(0xffffffffu, l[h], 2);
  }

  // ---- decode item: merge the four warps' partials in shared memory ----
  __syncthreads();  // every warp is done reading the K/V ring
  float* mbuf = reinterpret_cast<float*>(smem);  // [4 warps][16 rows][REC], over the idle ring
  if (compute) {
    float* mine = mbuf + warp * 16 * REC;
#pragma unroll
    for (int dn = 0; dn < DH / 8; ++dn) {
      const int col = dn * 8 + 2 * (lane & 3);
      mine[(lane >> 2) * REC + col] = oacc[dn][0];
      mine[(lane >> 2) * REC + col + 1] = oacc[dn][1];
      mine[((lane >> 2) + 8) * REC + col] = oacc[dn][2];
      mine[((lane >> 2) + 8) * REC + col + 1] = oacc[dn][3];
    }
    if ((lane & 3) == 0) {
      mine[(lane >> 2) * REC + DH] = m[0];
      mine[(lane >> 2) * REC + DH + 1] = l[0];
      mine[((lane >> 2) + 8) * REC + DH] = m[1];
      mine[((lane >> 2) + 8) * REC + DH + 1] = l[1];
    }
  }
  __syncthreads();
  const int tok = it.q_start;  // a decode segment has one row
  float* rec = p.part + static_cast<size_t>(it.part_base + it.split) * G * REC;
  for (int idx = tid; idx < G * DH; idx += ATT_THREADS) {
    const int g = idx / DH, d = idx - g * DH;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < 4; ++w) M = fmaxf(M, mbuf[(w * 16 + g) * REC + DH]);
    const float Ms = (M == -INFINITY) ? 0.0f : M;
    float L = 0.0f, o = 0.0f;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const float f = exp2f(mbuf[(w * 16 + g) * REC + DH] - Ms);
      L += mbuf[(w * 16 + g) * REC + DH + 1] * f;
      o += mbuf[(w * 16 + g) * REC + d] * f;
    }
    if (it.n_splits == 1) {
      p.out[(static_cast<size_t>(tok) * Hq + hk * G + g) * DH + d] = __float2half_rn(L > 0.0f ? o / L : 0.0f);
    } else {
      rec[g * REC + d] = o;
      if (d == 0) {
        rec[g * REC + DH] = M;
        rec[g * REC + DH + 1] = L;
      }
    }
  }
  if (it.n_splits == 1) return true;
  // ---- splits of this (row, kv head): the CTA that arrives last merges them in split order ----
  __threadfence();
  __syncthreads();
  uint32_t* counter = p.counters + it.seg * p.kv.Hkv + hk;
  if (tid == 0) {
    const uint32_t prev = atomicAdd(counter, 1u);
    is_last_s = (prev + 1u == static_cast<uint32_t>(it.n_splits)) ? 1u : 0u;
  }
  __syncthreads();
  if (!is_last_s) return true;
  __threadfence();
  const float* recs = p.part + static_cast<size_t>(it.part_base) * G * REC;
  for (int idx = tid; idx < G * DH; idx += ATT_THREADS) {
    const int g = idx / DH, d = idx - g * DH;
    float M = -INFINITY;
    for (int sp = 0; sp < it.n_splits; ++sp) M = fmaxf(M, __ldcg(recs + (static_cast<size_t>(sp) * G + g) * REC + DH));
    const float Ms = (M == -INFINITY) ? 0.0f : M;
    float L = 0.0f, o = 0.0f;
    for (int sp = 0; sp < it.n_splits; ++sp) {
      const float* r = recs + (static_cast<size_t>(sp) * G + g) * REC;
      const float f = exp2f(__ldcg(r + DH) - Ms);
      L += __ldcg(r + DH + 1) * f;
      o += __ldcg(r + d) * f;
    }
    p.out[(static_cast<size_t>(tok) * Hq + hk * G + g) * DH + d] = __float2half_rn(L > 0.0f ? o / L : 0.0f);
  }
  if (tid == 0) *counter = 0u;  // ready for the next launch
  return true;
}

// Parameters of the decode items of one layer.
inline AttnParams make_params(hb_ctx* c, const KvGeom& kv, int layer) {
  AttnParams p;
  p.q = c->q;
  p.out = c->attn_out;
  p.kv = kv;
  p.layer = layer;
  p.items = c->dd.attn_items;
  p.pages = c->dd.pages;
  p.part = c->attn_part;
  p.counters = c->attn_counters;
  p.status = c->status;
  p.Hq = c->cfg.n_heads;
  p.G = c->cfg.n_heads / c->cfg.n_kv_heads;
  p.scale_log2 = 1.4426950408889634f / sqrtf(static_cast<float>(c->cfg.head_dim));
  return p;
}

}  // namespace hb_dec
