// Chunk-row attention on the tcgen05 tensor cores (Section 3.2 of the paper: embedding / prefill
// chunks attend causally over their own earlier chunks plus themselves).
//
// One CTA handles 128 query rows = (128 / G) consecutive tokens x the G query heads of one KV head
// (G = Hq / Hkv) of one chunk segment, against every key the rows may see, in tiles of 64 keys
// (4 KV pages).  192 threads:
//   warp 0    TMA: gathers the pages of each key tile (one 2-D copy per page: the contiguous K+V
//             block of this KV head) into a shared-memory ring in the 128-byte-swizzled layout the
//             MMA descriptors expect
//   warp 1    MMA: S_j = Q K_j^T (128 x 64, fp32 in TMEM; Q is the A operand, held in TMEM) and
//             O += P_j V_j (128 x Dh, fp32 in TMEM), both tcgen05.mma kind::f16 from shared memory;
//             S_{j+1} is issued before P_j V_j so the tensor pipe works while softmax runs
//   warps 2-5 softmax: one thread per query row (TMEM lane): read its S row, mask, running max and
//             sum in fp32 (exp2), write P (fp16) to shared memory.  O stays in TMEM and is
//             rescaled only when a row's maximum grows by more than 2^8 since the maximum in use
//             (probabilities stay below 256, exact in fp16/fp32); the final 1/sum absorbs it.
// Every mbarrier wait is bounded; on expiry the CTA raises a status bit and leaves without
// storing.  The work split depends on the segment's own lengths only.
//
// This file is the body of one item; attention.cu includes it and calls it from the one attention
// kernel of the step, whose blocks stay resident and take one item after the other.  The block's
// 256 tensor-memory columns are allocated once by the kernel and handed in.
#pragma once
#include "hb_internal.h"
#include "ptx.cuh"

namespace hb_tc {

constexpr int TC_THREADS = 192;
constexpr int BM = 128;        // query rows per CTA
constexpr int BN = 64;         // keys per tile
constexpr uint64_t WAIT_NS = 1000000000ull;

struct TcParams {
  const __half* q;            // [T, Hq*Dh]
  __half* out;                // [T, Hq*Dh]
  int n_pages, Hkv, Hq, G, layer;
  const AttnItem* items;
  const int32_t* pages;
  uint32_t* status;
  float scale_log2;
};

template <int DH>
struct TcCfg {
  static constexpr int STAGES = (DH == 128) ? 3 : 4;
  static constexpr int KV_HALF = BN * DH * 2;            // K (or V) bytes of one stage
  static constexpr int PAGE_BYTES = DH * 64;             // one page block: [slot group][K|V][DH/64][8 keys][64]
  static constexpr int GROUP_BYTES = DH * 32;            // one slot group of a page block = stride of 8-key groups
  static constexpr int V_OFF = (DH / 64) * 1024;         // V part inside a slot group
  static constexpr int P_BYTES = BM * BN * 2;
  static constexpr int RING = STAGES * 2 * KV_HALF;
  static constexpr int BAR_OFF = RING + P_BYTES;
  static constexpr int TMEM_COLS = 256;
  static constexpr int S_COL = 0;                        // S: 64 columns (fp32)
  static constexpr int Q_COL = 64;                       // Q: DH/2 columns (two fp16 per column)
  static constexpr int O_COL = 128;                      // O: DH columns (fp32)
};

// Dynamic shared memory one chunk item needs.
template <int DH>
constexpr int smem_bytes() { return TcCfg<DH>::BAR_OFF + 8 * (2 * TcCfg<DH>::STAGES + 6) + 16; }

// The item's barrier words stop being barriers: the next item of the block may lay its shared memory
// out differently.  One thread, after the block has met at a barrier.
template <int DH>
__device__ __forceinline__ void retire_barriers(uint32_t smem_base) {
  for (int i = 0; i < 2 * TcCfg<DH>::STAGES + 6; ++i) mbar_inval(smem_base + TcCfg<DH>::BAR_OFF + 8u * i);
}

// One CTA of TC_THREADS threads, item `item` of p.items, with TcCfg::TMEM_COLS columns of tensor memory
// at `tmem`.  `kv_map` points at the kernel's __grid_constant__ tensor map.  Returns false (the same
// value in every thread) when the block must not take further items; *barriers_live tells whether
// retire_barriers is due.  `last_issue` is called once by thread 0 (the thread that talks to TMA) when
// it has requested the item's last key tile, i.e. a few tiles before the item ends (not on error paths).
template <int DH, class LastIssue>
__device__ __forceinline__ bool chunk_item(const CUtensorMap* kv_map, const TcParams& p, int item, uint32_t tmem,
                                           bool* barriers_live, LastIssue&& last_issue) {
  using C = TcCfg<DH>;
  extern __shared__ uint8_t smem_raw[];
  // The kernel has no static shared memory, so the dynamic window starts at the CTA's (1 KiB
  // aligned) shared-memory base, which the swizzled tiles need; checked, not assumed.
  const uint32_t base = smem_u32(smem_raw);
  uint8_t* smem = smem_raw;
  *barriers_live = false;
  if (base & 1023u) {
    if (threadIdx.x == 0) atomicOr(p.status, HB_DEV_ATTN_BAD_INDEX);
    return false;
  }
  const uint32_t ring_s = base, p_s = ring_s + C::RING, bar_s = base + C::BAR_OFF;
  auto kv_full = [&](int s) { return bar_s + 8u * s; };
  auto kv_empty = [&](int s) { return bar_s + 8u * (C::STAGES + s); };
  const uint32_t s_full = bar_s + 8u * (2 * C::STAGES), s_empty = bar_s + 8u * (2 * C::STAGES + 1);
  // P is handed over in two halves (keys 0-31, then 32-63) so that the first half of P V is issued
  // while the softmax threads are still producing the second
  const uint32_t q_ready = bar_s + 8u * (2 * C::STAGES + 2), p_ready2 = bar_s + 8u * (2 * C::STAGES + 3),
                 p_ready = bar_s + 8u * (2 * C::STAGES + 4), pv_done = bar_s + 8u * (2 * C::STAGES + 5);
  volatile uint32_t* abort_flag = reinterpret_cast<uint32_t*>(smem + C::BAR_OFF + 8 * (2 * C::STAGES + 6));

  const AttnItem it = p.items[item];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = p.G, Hq = p.Hq, hk = it.kv_head;
  const int n_tiles = (it.key1 + BN - 1) / BN;           // key0 is 0 for chunk items
  const int n_blk = (it.key1 + 15) / 16;

  if (tid == 0) {
    for (int s = 0; s < C::STAGES; ++s) { mbar_init(kv_full(s), 1); mbar_init(kv_empty(s), 1); }
    mbar_init(s_full, 1);
    mbar_init(s_empty, 4);
    mbar_init(q_ready, 4);
    mbar_init(p_ready, 4);
    mbar_init(p_ready2, 4);
    mbar_init(pv_done, 1);
    *abort_flag = 0u;
    mbar_init_fence();
  }
  // page ids are checked once here; the producer reads them from global memory as it goes
  int bad = 0;
  for (int i = tid; i < n_blk; i += TC_THREADS) {
    const int pg = (i < it.pt_len) ? p.pages[it.pt_start + i] : -1;
    bad |= (pg < 0 || pg >= p.n_pages);
  }
  *barriers_live = true;
  if (__syncthreads_or(bad)) {   // also publishes the barrier initialisation
    if (tid == 0) atomicOr(p.status, HB_DEV_ATTN_BAD_INDEX);
    return false;       // nothing requested from TMA
  }
  tc_fence_after();     // tensor-memory accesses of the block's previous item are ordered before this one's

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      // page ids of tile j + 1 are requested while tile j is being issued (global-load latency off the path)
      auto load_ids = [&](int j, int (&ids)[BN / 16]) {
        const int kb = j * BN;
#pragma unroll
        for (int pi = 0; pi < BN / 16; ++pi)
          ids[pi] = (kb + pi * 16 < it.key1) ? __ldg(p.pages + it.pt_start + kb / 16 + pi) : 0;
      };
      int nxt[BN / 16];
      load_ids(0, nxt);
      for (int j = 0; j < n_tiles; ++j) {
        const int st = j % C::STAGES;
        int cur[BN / 16];
#pragma unroll
        for (int pi = 0; pi < BN / 16; ++pi) cur[pi] = nxt[pi];
        if (j + 1 < n_tiles) load_ids(j + 1, nxt);
        if (!mbar_wait(kv_empty(st), static_cast<uint32_t>(((j / C::STAGES) & 1) ^ 1), abort_flag, WAIT_NS)) break;
        const int kb = j * BN;
        const int n_pg = min(BN / 16, (it.key1 - kb + 15) / 16);
        const uint32_t k_dst = ring_s + st * 2 * C::KV_HALF;
        mbar_arrive_expect_tx(kv_full(st), static_cast<uint32_t>(n_pg) * C::PAGE_BYTES);
#pragma unroll
        for (int pi = 0; pi < BN / 16; ++pi) {
          if (pi < n_pg) {
            const int64_t page = cur[pi];
            const int row = static_cast<int>(((static_cast<int64_t>(p.layer) * p.n_pages + page) * p.Hkv + hk) * (DH / 2));
            tma_load_2d(k_dst + pi * C::PAGE_BYTES, kv_map, kv_full(st), 0, row);   // K and V of this head, one copy
          }
        }
        if (j == n_tiles - 1) last_issue();
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      constexpr uint32_t idesc_s = make_idesc_f16(BM, BN, false);
      constexpr uint32_t idesc_o = make_idesc_f16(BM, DH, true);
      // S_j = Q K_j^T: Q comes from TMEM (written once by the softmax warps), K from shared memory: the
      // 8-key groups of the four page blocks of a tile are GROUP_BYTES apart, so one descriptor spans
      // all 64 keys.
      auto issue_s = [&](int j) -> bool {
        const int st = j % C::STAGES;
        if (!mbar_wait(kv_full(st), static_cast<uint32_t>((j / C::STAGES) & 1), abort_flag, WAIT_NS)) return false;
        if (!mbar_wait(s_empty, static_cast<uint32_t>((j & 1) ^ 1), abort_flag, WAIT_NS)) return false;
        tc_fence_after();
        const uint32_t k_tile = ring_s + st * 2 * C::KV_HALF;
#pragma unroll
        for (int ks = 0; ks < DH / 16; ++ks) {
          const uint64_t bd = make_desc(k_tile + (ks >> 2) * 1024 + (ks & 3) * 32, 16, C::GROUP_BYTES);
          umma_ts(tmem + static_cast<uint32_t>(C::S_COL), tmem + static_cast<uint32_t>(C::Q_COL + ks * 8), bd, idesc_s,
                  ks > 0 ? 1u : 0u);
        }
        umma_commit(s_full);
        return true;
      };
      bool ok = mbar_wait(q_ready, 0u, abort_flag, WAIT_NS);
      if (ok) ok = issue_s(0);
      for (int j = 0; ok && j < n_tiles; ++j) {
        // S_{j+1} may start as soon as the softmax warps have read S_j out of TMEM
        if (j + 1 < n_tiles) ok = issue_s(j + 1);
        if (!ok) break;
        const uint32_t kv_tile = ring_s + (j % C::STAGES) * 2 * C::KV_HALF;
        bool got = true;
#pragma unroll
        for (int ks = 0; ks < BN / 16; ++ks) {   // one page (16 keys = two 8-key groups) per k-step
          if (ks == 0 || ks == BN / 32) {        // each half of P has its own barrier
            if (!mbar_wait(ks == 0 ? p_ready : p_ready2, static_cast<uint32_t>(j & 1), abort_flag, WAIT_NS)) { got = false; break; }
            tc_fence_after();
          }
          const uint64_t ad = make_desc(p_s + ks * 32, 16, 1024);
          // V is the MN-major B operand: 64-column halves 1024 B apart, 8-key groups GROUP_BYTES apart
          const uint64_t bd = make_desc(kv_tile + ks * C::PAGE_BYTES + C::V_OFF, 1024, C::GROUP_BYTES);
          umma_ss(tmem + static_cast<uint32_t>(C::O_COL), ad, bd, idesc_o, (j > 0 || ks > 0) ? 1u : 0u);
        }
        if (!got) break;
        umma_commit(kv_empty(j % C::STAGES));
        umma_commit(pv_done);
      }
    }
    __syncwarp();
  } else {
    // ---------------- softmax (one thread per query row) ----------------
    const int quarter = warp & 3;
    const int rr = quarter * 32 + lane;                     // row of the tile = TMEM lane
    const bool row_valid = rr < it.n_rows;
    const int r = it.row0 + rr;
    const int pos = row_valid ? it.pos_start + r / G : -1;
    const uint32_t t_lane = tmem + (static_cast<uint32_t>(quarter * 32) << 16);
    float m_used = -INFINITY, l = 0.0f;
    bool ok = true;
    // the lanes of a warp leave the loop together (warp-wide votes and tcgen05.ld/st follow)
    auto wait_w = [&](uint32_t bar, uint32_t parity) {
      return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag, WAIT_NS)) != 0;
    };
    // this thread's query row -> TMEM (two fp16 per column), the A operand of every S MMA
    {
      const int tok = it.q_start + (row_valid ? r / G : 0), head = hk * G + (row_valid ? r % G : 0);
      const uint4* src = reinterpret_cast<const uint4*>(p.q + (static_cast<size_t>(tok) * Hq + head) * DH);
#pragma unroll
      for (int c = 0; c < DH / 2; c += 32) {
        uint32_t qr[32];
#pragma unroll
        for (int v = 0; v < 8; ++v) {
          const uint4 x = row_valid ? __ldg(src + c / 4 + v) : make_uint4(0u, 0u, 0u, 0u);
          qr[v * 4 + 0] = x.x; qr[v * 4 + 1] = x.y; qr[v * 4 + 2] = x.z; qr[v * 4 + 3] = x.w;
        }
        tmem_st32(t_lane + static_cast<uint32_t>(C::Q_COL + c), qr);
      }
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(q_ready);
    }
    for (int j = 0; j < n_tiles; ++j) {
      const int key_base = j * BN;
      if (!wait_w(s_full, static_cast<uint32_t>(j & 1))) { ok = false; break; }
      tc_fence_after();
      uint32_t sr[2][32];
      tmem_ld32(t_lane + static_cast<uint32_t>(C::S_COL), sr[0]);
      tmem_ld32(t_lane + static_cast<uint32_t>(C::S_COL + 32), sr[1]);
      tmem_ld_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(s_empty);
      // row maximum of the raw scores; masking only on tiles that touch the diagonal or the end of the keys
      const bool need_mask = (key_base + BN - 1 > pos) || (key_base + BN > it.key1);
      // (eight independent running maxima: a single chain of 64 dependent compares costs ~250 cycles
      // on a warp that has its scheduler to itself)
      float mx8[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) mx8[q] = -INFINITY;
      if (!need_mask) {
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
          for (int i = 0; i < 32; ++i) mx8[i & 7] = fmaxf(mx8[i & 7], __uint_as_float(sr[h][i]));
      } else {
        const int last = min(pos, it.key1 - 1) - key_base;   // last visible column of this row in the tile
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            if (h * 32 + i > last) sr[h][i] = 0xff800000u;   // -inf
            mx8[i & 7] = fmaxf(mx8[i & 7], __uint_as_float(sr[h][i]));
          }
      }
      float mx = fmaxf(fmaxf(fmaxf(mx8[0], mx8[1]), fmaxf(mx8[2], mx8[3])), fmaxf(fmaxf(mx8[4], mx8[5]), fmaxf(mx8[6], mx8[7])));
      mx *= p.scale_log2;   // scores enter the exponent as s * log2(e) / sqrt(Dh)
      const float m_new = fmaxf(m_used, mx);
      const bool grow = (m_new > m_used + 8.0f) || (m_used == -INFINITY && m_new > -INFINITY);
      // P_{j-1} V_{j-1} must have completed before O is rescaled or P is overwritten
      if (j > 0 && !wait_w(pv_done, static_cast<uint32_t>((j - 1) & 1))) { ok = false; break; }
      if (__any_sync(0xffffffffu, grow)) {
        const float f = grow ? exp2f(m_used - m_new) : 1.0f;   // m_used = -inf -> 0
        if (j > 0) {
          tc_fence_after();
#pragma unroll 1
          for (int c = 0; c < DH; c += 32) {
            uint32_t o[32];
            tmem_ld32(t_lane + static_cast<uint32_t>(C::O_COL + c), o);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * f);
            tmem_st32(t_lane + static_cast<uint32_t>(C::O_COL + c), o);
          }
          tmem_st_wait();
        }
        l *= f;
        if (grow) m_used = m_new;
      }
      const float neg_ms = (m_used == -INFINITY) ? 0.0f : -m_used;
      // probabilities p = 2^(s * scale - m) -> fp16 P row in shared memory (K-major, 128-byte swizzle)
      // keys past the end of the request hold stale bytes: zero those V rows (0 * garbage must stay 0)
      // before any part of P is handed over
      const int valid_keys = it.key1 - key_base;
      if (valid_keys < BN) {
        uint8_t* kv_gen = smem + (j % C::STAGES) * 2 * C::KV_HALF;
        const int t4 = tid - 64;  // 0..127 over the four softmax warps
        for (int u = t4; u < (BN - valid_keys) * (DH / 8); u += 128) {
          const int kr = valid_keys + u / (DH / 8), c = u % (DH / 8);
          *reinterpret_cast<uint4*>(kv_gen + (kr >> 4) * C::PAGE_BYTES + ((kr >> 3) & 1) * C::GROUP_BYTES + C::V_OFF +
                                    (c >> 3) * 1024 + (kr & 7) * 128 + (((c & 7) ^ (kr & 7)) << 4)) =
              make_uint4(0u, 0u, 0u, 0u);
        }
      }
      uint8_t* prow = smem + C::RING + rr * 128;
      float sum4[4] = {0.0f, 0.0f, 0.0f, 0.0f};   // fixed association, four short chains
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        uint32_t pk[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int i = c * 8 + e * 2;
          const float p0 = ex2_approx(fmaf(__uint_as_float(sr[i >> 5][i & 31]), p.scale_log2, neg_ms));
          const float p1 = ex2_approx(fmaf(__uint_as_float(sr[(i + 1) >> 5][(i + 1) & 31]), p.scale_log2, neg_ms));
          sum4[e] += p0 + p1;
          pk[e] = pack_half2(p0, p1);
        }
        *reinterpret_cast<uint4*>(prow + ((c ^ (rr & 7)) << 4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        if (c == 3 || c == 7) {   // keys 0-31 (then 32-63) of this warp's rows are in shared memory
          fence_async_smem();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(c == 3 ? p_ready : p_ready2);
        }
      }
      l += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
    }
    // ---- epilogue: O / l -> fp16 ----
    if (ok && n_tiles > 0 && wait_w(pv_done, static_cast<uint32_t>((n_tiles - 1) & 1))) {
      tc_fence_after();
      const float inv = (l > 0.0f) ? 1.0f / l : 0.0f;
      const int tok = it.q_start + (row_valid ? r / G : 0), head = hk * G + (row_valid ? r % G : 0);
      __half* orow = p.out + (static_cast<size_t>(tok) * Hq + head) * DH;
#pragma unroll 1
      for (int c = 0; c < DH; c += 32) {
        uint32_t o[32];
        tmem_ld32(t_lane + static_cast<uint32_t>(C::O_COL + c), o);
        tmem_ld_wait();
        if (row_valid) {
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            uint4 pk;
            pk.x = pack_half2(__uint_as_float(o[v * 8 + 0]) * inv, __uint_as_float(o[v * 8 + 1]) * inv);
            pk.y = pack_half2(__uint_as_float(o[v * 8 + 2]) * inv, __uint_as_float(o[v * 8 + 3]) * inv);
            pk.z = pack_half2(__uint_as_float(o[v * 8 + 4]) * inv, __uint_as_float(o[v * 8 + 5]) * inv);
            pk.w = pack_half2(__uint_as_float(o[v * 8 + 6]) * inv, __uint_as_float(o[v * 8 + 7]) * inv);
            *reinterpret_cast<uint4*>(orow + c + v * 8) = pk;
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  const bool aborted = (*abort_flag != 0u);
  if (aborted) {
    if (tid == 0) {
      atomicOr(p.status, HB_DEV_ATTN_WAIT_EXPIRED);
      for (int i = 0; i < 200; ++i) __nanosleep(1000);  // let requested copies land before the block goes on
    }
    __syncthreads();
  }
  return !aborted;
}

// Parameters of the chunk items of one layer.
inline TcParams make_params(hb_ctx* c, const KvGeom& kv, int layer) {
  TcParams p;
  p.q = c->q;
  p.out = c->attn_out;
  p.n_pages = kv.n_pages;
  p.Hkv = kv.Hkv;
  p.Hq = c->cfg.n_heads;
  p.G = c->cfg.n_heads / c->cfg.n_kv_heads;
  p.layer = layer;
  p.items = c->dd.tc_items;
  p.pages = c->dd.pages;
  p.status = c->status;
  p.scale_log2 = 1.4426950408889634f / sqrtf(static_cast<float>(c->cfg.head_dim));
  return p;
}

}  // namespace hb_tc
