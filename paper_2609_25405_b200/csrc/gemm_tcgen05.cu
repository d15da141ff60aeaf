// Projection GEMM for sm_100a: C = epilogue(A * B^T), A [M,K] fp16 activations and B [N,K] fp16 weights
// (the model's bf16 weights repacked once to fp16; tcgen05 kind::f16 needs one 16-bit format for both
// operands), both K-major, fp32 accumulation in tensor memory.
//
// These are the dense contractions of the shared forward pass (Section 3.1 of the paper:
// every row of the mixed batch goes through the same attention and feed-forward projections):
// QKV, O, gate/up, down and the LM head.
//
// Structure (one persistent CTA per SM, 320 threads):
//   warp 0   TMA producer: cp.async.bulk.tensor 2-D tiles (128B swizzle) into a ring of
//            shared-memory stages, completion on mbarriers
//   warp 1   MMA issuer: one thread issues tcgen05.mma (M=128, N=BN, K=16) from shared
//            memory descriptors into one of two TMEM accumulators; tcgen05.commit
//            releases stages and publishes finished accumulators
//   warps 2-9 epilogue: tcgen05.ld the accumulator (two warps per group of 32 TMEM lanes, half of
//            the tile's columns each), apply the epilogue, store with 16-byte vectors; overlaps
//            the next tile's main loop
// Two variants share the code.  CG = 1: one CTA per 128 x BN tile.  CG = 2: a cluster of two CTAs
// works on one 256 x 256 tile with tcgen05 cta_group::2: each CTA loads its own 128 rows of A and
// its own 128 rows of B (no multicast), the leader CTA issues MMAs that read both CTAs' shared
// memory, and each CTA's TMEM receives its 128 accumulator rows.  This halves the B traffic per SM
// and leaves room for six pipeline stages.
// Every mbarrier wait is bounded in time; on expiry the CTA raises a status bit, stops
// issuing work, lets outstanding copies land, frees its TMEM and returns.
#include "hb_internal.h"
#include "ptx.cuh"

namespace {

constexpr int BM = 128;
constexpr int BK = 64;
constexpr int UMMA_K = 16;
constexpr int NUM_THREADS = 320;   // TMA warp, MMA warp, eight epilogue warps
constexpr int EPI_WARPS = 8;
constexpr uint64_t WAIT_LIMIT_NS = 2000000000ull;  // 2 s

template <int BN, int CG>
struct Tile {
  static constexpr int B_ROWS = BN / CG;            // rows of B this CTA loads per stage
  static constexpr int STAGES = (B_ROWS == 256) ? 4 : 6;
  static constexpr int A_BYTES = BM * BK * 2;
  static constexpr int B_BYTES = B_ROWS * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int TMEM_COLS = (2 * BN <= 256) ? 256 : 512;  // two accumulators, rounded to a power of two
  static constexpr int BAR_BYTES = 256;
  // staging tiles of the residual epilogue: per epilogue warp 32 rows x 16 floats, rows 20 floats apart
  static constexpr int STG_PITCH = 20;
  static constexpr int STG_WARP_BYTES = 32 * STG_PITCH * 4;
  static constexpr int STG_OFF = STAGES * STAGE_BYTES + BAR_BYTES;
  static constexpr int SMEM_BYTES = STG_OFF + EPI_WARPS * STG_WARP_BYTES + 1024;  // + alignment slack
};

__device__ __forceinline__ float silu_f(float g) { return g / (1.0f + __expf(-g)); }

// Store one thread's 32 consecutive accumulator columns of one row.
template <int EPI>
__device__ __forceinline__ void epilogue_store(const GemmArgs& g, int row, int col0, const uint32_t (&r)[32]) {
  // col0 is a multiple of 32; N is a multiple of 8, so validity is decided per group of 8
  if constexpr (EPI == HB_EPI_F16) {
    __half* out = static_cast<__half*>(g.C) + static_cast<size_t>(row) * g.ldc + col0;
#pragma unroll
    for (int v = 0; v < 4; ++v) {
      if (col0 + v * 8 < g.N) {
        uint4 pk;
        pk.x = pack_half2_sat(__uint_as_float(r[v * 8 + 0]), __uint_as_float(r[v * 8 + 1]));
        pk.y = pack_half2_sat(__uint_as_float(r[v * 8 + 2]), __uint_as_float(r[v * 8 + 3]));
        pk.z = pack_half2_sat(__uint_as_float(r[v * 8 + 4]), __uint_as_float(r[v * 8 + 5]));
        pk.w = pack_half2_sat(__uint_as_float(r[v * 8 + 6]), __uint_as_float(r[v * 8 + 7]));
        *reinterpret_cast<uint4*>(out + v * 8) = pk;
      }
    }
  } else if constexpr (EPI == HB_EPI_LORA_DOWN) {
    // rank-r activations of the adapted rows: alpha * acc for rows >= first_row, zero for the rows
    // before it (rows of request kinds that do not carry the adapter)
    __half* out = static_cast<__half*>(g.C) + static_cast<size_t>(row) * g.ldc + col0;
    const float a = (row >= g.first_row) ? g.alpha : 0.0f;
#pragma unroll
    for (int v = 0; v < 4; ++v) {
      if (col0 + v * 8 < g.N) {
        uint4 pk;
        pk.x = pack_half2_sat(a * __uint_as_float(r[v * 8 + 0]), a * __uint_as_float(r[v * 8 + 1]));
        pk.y = pack_half2_sat(a * __uint_as_float(r[v * 8 + 2]), a * __uint_as_float(r[v * 8 + 3]));
        pk.z = pack_half2_sat(a * __uint_as_float(r[v * 8 + 4]), a * __uint_as_float(r[v * 8 + 5]));
        pk.w = pack_half2_sat(a * __uint_as_float(r[v * 8 + 6]), a * __uint_as_float(r[v * 8 + 7]));
        *reinterpret_cast<uint4*>(out + v * 8) = pk;
      }
    }
  } else if constexpr (EPI == HB_EPI_F32 || EPI == HB_EPI_RESID_F32) {
    float* out = static_cast<float*>(g.C) + static_cast<size_t>(row) * g.ldc + col0;
#pragma unroll
    for (int v = 0; v < 8; ++v) {
      if (col0 + v * 4 < g.N) {
        float4 o;
        o.x = __uint_as_float(r[v * 4 + 0]);
        o.y = __uint_as_float(r[v * 4 + 1]);
        o.z = __uint_as_float(r[v * 4 + 2]);
        o.w = __uint_as_float(r[v * 4 + 3]);
        if constexpr (EPI == HB_EPI_RESID_F32) {
          // (plain load: with split K these rows were written earlier in this launch, by another SM
          // whose stores went to L2, or by this SM itself; this SM's L1 holds no older copy of them)
          const float4 old = *reinterpret_cast<const float4*>(out + v * 4);
          o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w;
        }
        *reinterpret_cast<float4*>(out + v * 4) = o;
      }
    }
  } else {  // HB_EPI_SWIGLU: columns (2j, 2j+1) = (gate_j, up_j) -> out column j
    __half* out = static_cast<__half*>(g.C) + static_cast<size_t>(row) * g.ldc + col0 / 2;
#pragma unroll
    for (int v = 0; v < 2; ++v) {
      if (col0 + v * 16 < g.N) {
        uint32_t pk[4];
        bool range = false;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float g0 = __uint_as_float(r[v * 16 + j * 4 + 0]), u0 = __uint_as_float(r[v * 16 + j * 4 + 1]);
          const float g1 = __uint_as_float(r[v * 16 + j * 4 + 2]), u1 = __uint_as_float(r[v * 16 + j * 4 + 3]);
          const float a0 = silu_f(g0) * u0, a1 = silu_f(g1) * u1;
          range |= outside_half_range(a0) | outside_half_range(a1);
          pk[j] = pack_half2_sat(a0, a1);
        }
        *reinterpret_cast<uint4*>(out + v * 8) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        // the FFN's inner activation is the widest-ranging fp16 value of the step: report, do not hide
        if (range) atomicOr(g.status, HB_DEV_F16_RANGE);
      }
    }
  }
}

// Residual update x += acc for one 32 x 32 block (this warp's 32 rows, 32 columns from col0).  In
// TMEM a thread owns a row, so storing straight from registers makes every warp-level access touch
// 32 different rows (one 16-byte piece of 32 cache lines), and with each load of x followed by its
// store the compiler has to keep every load behind the previous store (they could alias): measured
// 44-49 k cycles per 256 x 256 tile, longer than the 64-k-block main loop it should hide behind.
// The block goes through a shared-memory tile instead, 16 columns at a time, and comes back with
// four lanes per row (64-byte row segments of eight rows per access); all loads of x are issued
// before the first store.
__device__ __forceinline__ void resid_block_store(const GemmArgs& g, float* stg, int pitch, int lane, int row0,
                                                  int col0, const uint32_t (&r)[32]) {
  float* mine = stg + lane * pitch;
  const int sub = lane >> 2, cq = (lane & 3) * 4;
#pragma unroll
  for (int hcol = 0; hcol < 2; ++hcol) {
#pragma unroll
    for (int v = 0; v < 4; ++v)
      *reinterpret_cast<float4*>(mine + v * 4) =
          make_float4(__uint_as_float(r[hcol * 16 + v * 4 + 0]), __uint_as_float(r[hcol * 16 + v * 4 + 1]),
                      __uint_as_float(r[hcol * 16 + v * 4 + 2]), __uint_as_float(r[hcol * 16 + v * 4 + 3]));
    __syncwarp();
    const int cb = col0 + hcol * 16 + cq;
    if (cb < g.N) {   // N is a multiple of 8: a group of four columns is valid or not as a whole
      float* base = static_cast<float*>(g.C) + static_cast<size_t>(row0 + sub) * g.ldc + cb;
      float4 old[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        // (plain load: with split K these rows were written earlier in this launch, by another SM
        // whose stores went to L2, or by this SM itself; this SM's L1 holds no older copy of them)
        if (row0 + i * 8 + sub < g.M) old[i] = *reinterpret_cast<const float4*>(base + static_cast<size_t>(i) * 8 * g.ldc);
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        if (row0 + i * 8 + sub < g.M) {
          const float4 a = *reinterpret_cast<const float4*>(stg + (i * 8 + sub) * pitch + cq);
          *reinterpret_cast<float4*>(base + static_cast<size_t>(i) * 8 * g.ldc) =
              make_float4(old[i].x + a.x, old[i].y + a.y, old[i].z + a.z, old[i].w + a.w);
        }
      }
    }
    __syncwarp();   // the tile may be rewritten
  }
}

// Split-K partial of the thin adapter GEMM: fp32, [split][row][N].
__device__ __forceinline__ void store_partial(const GemmArgs& g, int split, int row, int col0, const uint32_t (&r)[32]) {
  float* out = g.split_part + (static_cast<size_t>(split) * g.M + row) * g.N + col0;
#pragma unroll
  for (int v = 0; v < 8; ++v) {
    if (col0 + v * 4 < g.N)
      *reinterpret_cast<float4*>(out + v * 4) = make_float4(__uint_as_float(r[v * 4 + 0]), __uint_as_float(r[v * 4 + 1]),
                                                             __uint_as_float(r[v * 4 + 2]), __uint_as_float(r[v * 4 + 3]));
  }
}

// QKV epilogue: one thread holds 32 consecutive output columns of one token row.  The q and k rows
// of the weight are pair-interleaved inside each head (column 2i = rotary element i, column 2i+1 =
// element i + Dh/2), so every rotation pair sits in adjacent columns.  q goes to the query buffer,
// k and v to slot pos % P of the row's page; all as fp16.
// Address of 32 consecutive head-dimension elements starting at `off` of one cache row.  Arena layout:
// [page][kv head][slot group (slots 0-7 | 8-15)][K|V][Dh/64 halves][8 slots][64]: the K+V block of one
// (page, head) is contiguous (one TMA copy), and the 8-row groups of K (or V) of consecutive pages
// landed back to back in shared memory are a uniform stride apart, as the MMA descriptors need.
__device__ __forceinline__ __half* kv_slot_ptr(const GemmArgs& g, int page, int kv_head, int is_v, int slot, int off) {
  const int halves = g.Dh >> 6;
  return g.kv_layer + static_cast<int64_t>(page) * g.page_stride + static_cast<int64_t>(kv_head) * 2 * g.Dh * g.P +
         (slot >> 3) * (g.Dh * g.P) + (is_v * halves + (off >> 6)) * 512 + (slot & 7) * 64 + (off & 63);
}

__device__ __forceinline__ void epilogue_qkv_rope(const GemmArgs& g, int row, int col0, const uint32_t (&r)[32],
                                                  int pos, int page) {
  const int Dh = g.Dh;
  const int head = col0 / Dh, off = col0 - head * Dh;
  uint32_t pk[16];
  __half* dst;
  if (head < g.Hq + g.Hkv) {
    const float4* cs = reinterpret_cast<const float4*>(g.rope_cos + static_cast<size_t>(pos) * (Dh >> 1) + (off >> 1));
    const float4* sn = reinterpret_cast<const float4*>(g.rope_sin + static_cast<size_t>(pos) * (Dh >> 1) + (off >> 1));
#pragma unroll
    for (int v = 0; v < 4; ++v) {
      const float4 c = __ldg(cs + v), s = __ldg(sn + v);
      const float cc[4] = {c.x, c.y, c.z, c.w}, ss[4] = {s.x, s.y, s.z, s.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float a = __uint_as_float(r[v * 8 + e * 2]), b = __uint_as_float(r[v * 8 + e * 2 + 1]);
        pk[v * 4 + e] = pack_half2_sat(a * cc[e] - b * ss[e], b * cc[e] + a * ss[e]);
      }
    }
    if (head < g.Hq) {
      dst = g.q_out + static_cast<size_t>(row) * g.Hq * Dh + col0;
    } else {
      dst = kv_slot_ptr(g, page, head - g.Hq, 0, pos % g.P, off);
    }
  } else {
#pragma unroll
    for (int j = 0; j < 16; ++j) pk[j] = pack_half2_sat(__uint_as_float(r[2 * j]), __uint_as_float(r[2 * j + 1]));
    dst = kv_slot_ptr(g, page, head - g.Hq - g.Hkv, 1, pos % g.P, off);
  }
#pragma unroll
  for (int v = 0; v < 4; ++v)
    *reinterpret_cast<uint4*>(dst + v * 8) = make_uint4(pk[v * 4], pk[v * 4 + 1], pk[v * 4 + 2], pk[v * 4 + 3]);
}

template <int BN, int EPI, int CG>
__global__ void __launch_bounds__(NUM_THREADS, 1)
hb_gemm_tcgen05_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                       const __grid_constant__ CUtensorMap tmA2, const __grid_constant__ CUtensorMap tmB2,
                       const GemmArgs g) {
  using T = Tile<BN, CG>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t bar_base = smem_base + T::STAGES * T::STAGE_BYTES;
  // barrier layout (8 B each): full[STAGES], empty[STAGES], tfull[2], tempty[2]; then tmem slot, abort flag
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (T::STAGES + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * T::STAGES + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * T::STAGES + 2 + a); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_gen + T::STAGES * T::STAGE_BYTES + 8 * (2 * T::STAGES + 4));
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  // CG = 2: the two CTAs of a cluster share every tile; rank 0 leads (issues the MMAs and owns
  // the full / tmem-empty barriers).  CG = 1: every CTA is its own leader.
  const uint32_t rank = (CG == 2) ? cluster_ctarank() : 0u;
  const bool leader = (rank == 0u);
  const int worker = (CG == 2) ? static_cast<int>(blockIdx.x >> 1) : static_cast<int>(blockIdx.x);
  const int n_workers = (CG == 2) ? static_cast<int>(gridDim.x >> 1) : static_cast<int>(gridDim.x);

  const int m_tiles = (g.M + BM * CG - 1) / (BM * CG);
  const int n_tiles = (g.N + BN - 1) / BN;
  // k_splits > 1: every output tile is computed by k_splits work items, each over an equal share of
  // the K blocks.  Thin adapter GEMMs merge fp32 partials in split order; residual-update GEMMs add
  // their shares to x one after the other, split s after split s - 1 (a fixed order, so a row's
  // result does not depend on timing or on the batch).  Items are ordered split-major: every
  // split-0 item precedes every split-1 item, and a worker takes its items in increasing order, so
  // the item a waiting epilogue depends on is never queued behind an item that itself waits.
  const int mn_tiles = m_tiles * n_tiles;
  const int k_splits = (EPI == HB_EPI_LORA_DOWN || EPI == HB_EPI_RESID_F32) ? max(g.k_splits, 1) : 1;
  const int total_tiles = mn_tiles * k_splits;
  // K runs over the columns of (A, B) and then over g.k2_blocks more 64-column blocks of a second
  // operand pair (A2, B2): C = A B^T + A2 B2^T in one accumulation (the low-rank branch of an
  // adapted projection, with A2 = the rows' rank-r activations and B2 = the up factor).
  const int k1_blocks = (g.K + BK - 1) / BK;
  const int k_blocks = k1_blocks + g.k2_blocks;
  // Splits share the main K blocks evenly; the second pair's blocks all go to the last split, so
  // that where a row's sum is cut does not depend on whether the launch carries a second pair (a
  // generation row's bits must not change when embedding rows with an adapter join its batch).
  const int k_per_split = (k1_blocks + k_splits - 1) / k_splits;
  // Tile walk: output tiles are numbered along M first inside bands of `band` row tiles, band after
  // band.  With band = m_tiles this is "rows fastest over the whole M" (a wave of workers touches every
  // row tile of A and a few column tiles of B).  When A's share of a work item is too large for all its
  // row tiles to stay in L2 next to the B tiles streaming past, a narrower band keeps the band's rows
  // of A resident while the walk crosses N, at the price of one more pass over B per band.  The walk
  // changes which worker computes a tile and when, never the order of the K sum of an element.
  const int band = (g.raster_band > 0 && g.raster_band < m_tiles) ? g.raster_band : m_tiles;
  auto tile_coords = [&](int mn, int& mi, int& ni) {
    const int per_band = band * n_tiles;
    const int b = mn / per_band, r = mn - b * per_band;
    const int bh = min(band, m_tiles - b * band);
    ni = r / bh;
    mi = b * band + (r - ni * bh);
  };

  if (threadIdx.x == 0) {
    for (int s = 0; s < T::STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tfull_bar(a), 1);
      mbar_init(tempty_bar(a), EPI_WARPS * CG);  // one arrival per epilogue warp of every CTA of the group
    }
    *abort_flag = 0u;
    mbar_init_fence();
  }
  if (warp == 1) {
    if constexpr (CG == 2) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                   "r"(static_cast<uint32_t>(T::TMEM_COLS))
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                   "r"(static_cast<uint32_t>(T::TMEM_COLS))
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  __syncthreads();
  if constexpr (CG == 2) cluster_sync();  // the peer's barriers are initialised before anything signals them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // Everything above touches only this CTA's shared memory and TMEM, so it may run while the previous
  // kernel of the stream drains.  The order "allocate, wait, let the next kernel in" means that when a
  // following kernel's CTAs become resident every CTA of this one already holds its TMEM columns.
  grid_dep_wait();
  grid_dep_launch();

  // Give up: raise the flag here and in the peer CTA so that every role of the group leaves its loop.
  auto give_up = [&]() {
    *abort_flag = 1u;
    if constexpr (CG == 2) st_cluster_u32(map_to_rank(smem_u32(const_cast<uint32_t*>(abort_flag)), rank ^ 1u), 1u);
  };

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      const uint64_t pol_a = g.l2_hints ? l2_policy_evict_last() : 0ull;
      const uint64_t pol_b = g.l2_hints ? l2_policy_evict_first() : 0ull;
      // the data of both CTAs of a group is accounted on the leader's barrier
      for (int tile = worker; ok && tile < total_tiles; tile += n_workers) {
        const int mn = tile % mn_tiles, split = tile / mn_tiles;
        int mi, ni;
        tile_coords(mn, mi, ni);
        const int m0 = mi * (BM * CG) + static_cast<int>(rank) * BM;
        const int n0 = ni * BN + static_cast<int>(rank) * T::B_ROWS;
        const int kb0 = split * k_per_split;
        const int kb1 = (split + 1 == k_splits) ? k_blocks : min(kb0 + k_per_split, k1_blocks);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, WAIT_LIMIT_NS)) { ok = false; give_up(); break; }
          const uint32_t a_dst = smem_base + stage * T::STAGE_BYTES;
          const uint32_t b_dst = a_dst + T::A_BYTES;
          const bool ext = (kb >= k1_blocks);
          const CUtensorMap* ma = ext ? &tmA2 : &tmA;
          const CUtensorMap* mb = ext ? &tmB2 : &tmB;
          const int ka = ext ? (kb - k1_blocks) * BK : kb * BK;
          const int kbb = ext ? ka : (kb >> g.b_kshift) * BK;
          if constexpr (CG == 2) {
            const uint32_t bar = map_to_rank(full_bar(stage), 0u);
            if (leader) mbar_arrive_expect_tx(full_bar(stage), 2u * T::STAGE_BYTES);
            if (g.l2_hints) {
              tma_load_2d_cg2_hint(a_dst, ma, bar, ka, m0, pol_a);
              tma_load_2d_cg2_hint(b_dst, mb, bar, kbb, n0, pol_b);
            } else {
              tma_load_2d_cg2(a_dst, ma, bar, ka, m0);
              tma_load_2d_cg2(b_dst, mb, bar, kbb, n0);
            }
          } else {
            mbar_arrive_expect_tx(full_bar(stage), T::STAGE_BYTES);
            if (g.l2_hints) {
              tma_load_2d_hint(a_dst, ma, full_bar(stage), ka, m0, pol_a);
              tma_load_2d_hint(b_dst, mb, full_bar(stage), kbb, n0, pol_b);
            } else {
              tma_load_2d(a_dst, ma, full_bar(stage), ka, m0);
              tma_load_2d(b_dst, mb, full_bar(stage), kbb, n0);
            }
          }
          if (++stage == T::STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        // give copies already in flight time to land before shared memory is released
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ---------------- MMA issuer (leader CTA only) ----------------
    if (lane == 0 && leader) {
      constexpr uint32_t idesc = make_idesc_f16(BM * CG, BN, false);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int tile = worker; ok && tile < total_tiles; tile += n_workers) {
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, WAIT_LIMIT_NS)) { ok = false; give_up(); break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * BN);
        const int split = tile / mn_tiles;
        const int kb0 = split * k_per_split;
        const int kb1 = (split + 1 == k_splits) ? k_blocks : min(kb0 + k_per_split, k1_blocks);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag, WAIT_LIMIT_NS)) { ok = false; give_up(); break; }
          tc_fence_after();
          const uint32_t a_addr = smem_base + stage * T::STAGE_BYTES;
          const uint64_t adesc = make_desc(a_addr, 16, 1024);
          const uint64_t bdesc = make_desc(a_addr + T::A_BYTES, 16, 1024);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            // advancing 16 elements along K inside the 128-byte swizzle row = +32 B = +2 in the address field
            const uint32_t accum = (kb > kb0 || k > 0) ? 1u : 0u;
            if constexpr (CG == 2) umma_ss_cg2(d_tmem, adesc + 2u * k, bdesc + 2u * k, idesc, accum);
            else umma_ss(d_tmem, adesc + 2u * k, bdesc + 2u * k, idesc, accum);
          }
          // the stage is free (in every CTA of the group) once these MMAs have read it
          if constexpr (CG == 2) umma_commit_cg2(empty_bar(stage));
          else umma_commit(empty_bar(stage));
          if (++stage == T::STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        if constexpr (CG == 2) umma_commit_cg2(tfull_bar(acc));  // accumulator complete (both CTAs)
        else umma_commit(tfull_bar(acc));
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
    __syncwarp();
  } else {
    // ---------------- epilogue (warps 2..9) ----------------
    // Two warps share each group of 32 TMEM lanes (rows): warps 2-5 take the left half of the tile's
    // columns, warps 6-9 the right half, so a tile's epilogue - and with it the one after a CTA's
    // last tile, which nothing hides - takes half as long.
    const int quarter = warp & 3;  // TMEM lanes [32*quarter, 32*quarter + 32) belong to this warp
    const int half = (warp - 2) >> 2;
    const int epi_slot = half * 4 + quarter;   // 0..7
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int tile = worker; ok && tile < total_tiles; tile += n_workers) {
      const int mn = tile % mn_tiles, split = tile / mn_tiles;
      int mi, ni;
      tile_coords(mn, mi, ni);
      const int m0 = mi * (BM * CG) + static_cast<int>(rank) * BM;
      const int n0 = ni * BN;
      if (!mbar_wait(tfull_bar(acc), acc_phase, abort_flag, WAIT_LIMIT_NS)) { ok = false; give_up(); break; }
      tc_fence_after();
      const int row = m0 + quarter * 32 + lane;
      const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + static_cast<uint32_t>(acc * BN);
      int pos = 0, page = 0;
      bool row_ok = row < g.M;
      if constexpr (EPI == HB_EPI_QKV_ROPE) {
        if (row_ok) {
          pos = g.row_pos[row];
          page = g.row_page[row];
          if (page < 0 || page >= g.n_pages) {   // never write through a bad page id
            atomicOr(g.status, HB_DEV_APPEND_BAD_INDEX);
            row_ok = false;
          }
        }
      }
      uint32_t* turn = nullptr;
      if constexpr (EPI == HB_EPI_RESID_F32) {
        if (k_splits > 1) {
          // one turn word per (tile, CTA of the group, warp): these 32 rows of the tile are updated by
          // split 0, then split 1, ...; the word holds the split whose turn it is
          turn = g.split_counters + ((static_cast<size_t>(mn) * CG + rank) * EPI_WARPS + epi_slot);
          if (split > 0) {
            uint32_t okw = 1u;
            if (lane == 0) {
              const uint64_t t0 = global_ns();
              while (ld_acquire_u32(turn) != static_cast<uint32_t>(split)) {
                if (*abort_flag || global_ns() - t0 > WAIT_LIMIT_NS) { okw = 0u; break; }
                __nanosleep(64);
              }
            }
            okw = __shfl_sync(0xffffffffu, okw, 0);
            if (!okw) { ok = false; give_up(); break; }
          }
        }
      }
#pragma unroll 1
      for (int c = half * (BN / 2); c < (half + 1) * (BN / 2); c += 32) {
        uint32_t r[32];
        tmem_ld32(t_row + static_cast<uint32_t>(c), r);
        tmem_ld_wait();
        if constexpr (EPI == HB_EPI_RESID_F32) {
          // every lane takes part (the block is exchanged through shared memory); rows and columns
          // past the edges are masked inside
          if (n0 + c < g.N)
            resid_block_store(g, reinterpret_cast<float*>(smem_gen + T::STG_OFF + epi_slot * T::STG_WARP_BYTES),
                              T::STG_PITCH, lane, m0 + quarter * 32, n0 + c, r);
        } else if (row_ok && n0 + c < g.N) {
          if constexpr (EPI == HB_EPI_QKV_ROPE) {
            epilogue_qkv_rope(g, row, n0 + c, r, pos, page);
          } else if constexpr (EPI == HB_EPI_LORA_DOWN) {
            if (k_splits > 1) store_partial(g, split, row, n0 + c, r);
            else epilogue_store<EPI>(g, row, n0 + c, r);
          } else {
            epilogue_store<EPI>(g, row, n0 + c, r);
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if constexpr (CG == 2) mbar_arrive_cluster(map_to_rank(tempty_bar(acc), 0u));
        else mbar_arrive(tempty_bar(acc));
      }
      if constexpr (EPI == HB_EPI_RESID_F32) {
        if (turn != nullptr) {
          // this warp's rows of x are written: pass the turn on (the last split leaves the word at 0
          // for the next launch)
          __threadfence();
          __syncwarp();
          if (lane == 0) st_release_u32(turn, split + 1 == k_splits ? 0u : static_cast<uint32_t>(split + 1));
        }
      }
      if constexpr (EPI == HB_EPI_LORA_DOWN) {
        if (k_splits > 1) {
          // The warp that arrives last for these 32 rows of the tile adds the partial sums in split
          // order (a fixed order: the result does not depend on which work item finished when).
          __threadfence();
          __syncwarp();
          uint32_t prev = 0;
          uint32_t* ctr = g.split_counters + (static_cast<size_t>(mn) * EPI_WARPS + epi_slot);
          if (lane == 0) prev = atomicAdd(ctr, 1u);
          prev = __shfl_sync(0xffffffffu, prev, 0);
          if (prev + 1u == static_cast<uint32_t>(k_splits)) {
            __threadfence();
            if (row_ok) {
              for (int c = half * (BN / 2); c < (half + 1) * (BN / 2) && n0 + c < g.N; c += 32) {
                uint32_t r[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) r[j] = 0u;   // +0.0f
                for (int sp = 0; sp < k_splits; ++sp) {
                  const float* src = g.split_part + (static_cast<size_t>(sp) * g.M + row) * g.N + n0 + c;
#pragma unroll
                  for (int v = 0; v < 8; ++v) {
                    if (n0 + c + v * 4 < g.N) {
                      const float4 p = __ldcg(reinterpret_cast<const float4*>(src + v * 4));
                      r[v * 4 + 0] = __float_as_uint(__uint_as_float(r[v * 4 + 0]) + p.x);
                      r[v * 4 + 1] = __float_as_uint(__uint_as_float(r[v * 4 + 1]) + p.y);
                      r[v * 4 + 2] = __float_as_uint(__uint_as_float(r[v * 4 + 2]) + p.z);
                      r[v * 4 + 3] = __float_as_uint(__uint_as_float(r[v * 4 + 3]) + p.w);
                    }
                  }
                }
                epilogue_store<EPI>(g, row, n0 + c, r);
              }
            }
            __syncwarp();
            if (lane == 0) *ctr = 0u;   // ready for the next launch
          }
        }
      }
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  }

  tc_fence_before();
  __syncthreads();
  // no CTA of a group leaves (or frees TMEM) while its peer may still read its shared memory or signal it
  if constexpr (CG == 2) cluster_sync();
  if (threadIdx.x == 0 && *abort_flag) atomicOr(g.status, HB_DEV_GEMM_WAIT_EXPIRED);
  if (warp == 1) {
    tc_fence_after();
    if constexpr (CG == 2)
      asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                   "r"(static_cast<uint32_t>(T::TMEM_COLS))
                   : "memory");
    else
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                   "r"(static_cast<uint32_t>(T::TMEM_COLS))
                   : "memory");
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

template <int BN, int EPI, int CG>
int launch_one(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmA2, const CUtensorMap& tmB2,
               const GemmArgs& a, int num_sms, cudaStream_t s, bool pdl) {
  using T = Tile<BN, CG>;
  static DynSmemState configured;   // per device: a second GPU in the process needs the attribute too
  auto kern = hb_gemm_tcgen05_kernel<BN, EPI, CG>;
  if (hb_ensure_dyn_smem(reinterpret_cast<const void*>(kern), configured, T::SMEM_BYTES) != HB_OK) return HB_ERR_CUDA;
  const int m_tiles = (a.M + BM * CG - 1) / (BM * CG);
  const int n_tiles = (a.N + BN - 1) / BN;
  int workers = m_tiles * n_tiles *
                (((EPI == HB_EPI_LORA_DOWN || EPI == HB_EPI_RESID_F32) && a.k_splits > 1) ? a.k_splits : 1);
  if (workers > num_sms / CG) workers = num_sms / CG;
  if (workers < 1) return HB_OK;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(workers * CG));
  cfg.blockDim = dim3(NUM_THREADS);
  cfg.dynamicSmemBytes = T::SMEM_BYTES;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CG;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, kern, tmA, tmB, tmA2, tmB2, a) == cudaSuccess ? HB_OK : HB_ERR_CUDA;
}

template <int BN, int CG>
int launch_bn(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmA2, const CUtensorMap& tmB2,
              int epi, const GemmArgs& a, int num_sms, cudaStream_t s, bool pdl) {
  switch (epi) {
    case HB_EPI_F16: return launch_one<BN, HB_EPI_F16, CG>(tmA, tmB, tmA2, tmB2, a, num_sms, s, pdl);
    case HB_EPI_F32: return launch_one<BN, HB_EPI_F32, CG>(tmA, tmB, tmA2, tmB2, a, num_sms, s, pdl);
    case HB_EPI_RESID_F32: return launch_one<BN, HB_EPI_RESID_F32, CG>(tmA, tmB, tmA2, tmB2, a, num_sms, s, pdl);
    case HB_EPI_SWIGLU: return launch_one<BN, HB_EPI_SWIGLU, CG>(tmA, tmB, tmA2, tmB2, a, num_sms, s, pdl);
    case HB_EPI_QKV_ROPE: return launch_one<BN, HB_EPI_QKV_ROPE, CG>(tmA, tmB, tmA2, tmB2, a, num_sms, s, pdl);
    case HB_EPI_LORA_DOWN:
      if constexpr (CG == 1) return launch_one<BN, HB_EPI_LORA_DOWN, CG>(tmA, tmB, tmA2, tmB2, a, num_sms, s, pdl);
      else return HB_ERR_BAD_ARG;
    default: return HB_ERR_BAD_ARG;
  }
}

}  // namespace

int hb_tmap_2d_f16(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  EncodeTiledFn enc = get_encode_fn();
  if (!enc) return HB_ERR_CUDA;
  if ((reinterpret_cast<uintptr_t>(base) & 15u) || (cols & 7u) || rows == 0 || cols == 0) return HB_ERR_BAD_ARG;
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * 2};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(BK), box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(base), dims, strides, box,
                         estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                         CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? HB_OK : HB_ERR_CUDA;
}

// Tile width: 256 columns halves the shared-memory traffic per flop; 128 gives more tiles
// when the problem has too few to fill the SMs or the last wave would be mostly idle.
int hb_gemm_pick_bn(int M, int N, int num_sms) {
  // enough rows and columns for 256 x 256 pair tiles to fill the machine: use CTA pairs.  (A 256 x 192
  // pair tile would shorten the last, partly filled wave of the N = 4096 and 6144 projections, but it
  // measured 10-19 % slower on every 7B shape: the kernel is bound by bytes loaded per MMA cycle,
  // which the narrower tile raises.)
  if (M > 128 && static_cast<long>((M + 255) / 256) * ((N + 255) / 256) >= num_sms / 2) return HB_GEMM_PAIR256;
  const int m_tiles = (M + BM - 1) / BM;
  const long t256 = static_cast<long>(m_tiles) * ((N + 255) / 256);
  const long t128 = static_cast<long>(m_tiles) * ((N + 127) / 128);
  if (t256 < num_sms) return 128;
  const double e256 = static_cast<double>(t256) / (((t256 + num_sms - 1) / num_sms) * num_sms);
  const double e128 = static_cast<double>(t128) / (((t128 + num_sms - 1) / num_sms) * num_sms);
  return (e128 * 0.92 > e256) ? 128 : 256;
}

// Residual-update GEMMs may split K in two when that fills the last wave of CTA pairs much better
// (7B shape at 4096 rows: 256 tiles on 74 pairs is 3.46 waves, 512 half-K items is 6.92).  The choice
// depends on the problem shape alone, never on the batch at hand.
int hb_gemm_pick_ksplit(int M, int N, int K, int variant, int num_sms) {
  if (variant != HB_GEMM_PAIR256) return 1;
  const long workers = num_sms / 2;
  // each half must still be long enough to hide an epilogue that reads and writes the whole tile
  if (workers < 1 || K < 128 * BK) return 1;
  const long tiles = static_cast<long>((M + 255) / 256) * ((N + 255) / 256);
  const double e1 = static_cast<double>(tiles) / (((tiles + workers - 1) / workers) * workers);
  const double e2 = static_cast<double>(2 * tiles) / (((2 * tiles + workers - 1) / workers) * workers);
  return e2 > e1 * 1.05 ? 2 : 1;
}

// CTA-pair 256 x 256 tiles and single-CTA 128 x 128 tiles read B through the same 128-row boxes and
// accumulate every output element over K in the same order, so their results are bit-identical
// (checked in the tests) and a launch may use whichever is faster for its own row count without a
// request's result depending on its batch.  K splits are not part of this choice: they change the
// summation order and stay fixed per context.  The estimate is waves x time per wave with figures
// measured on the 1B- and 7B-class projections (microseconds; k = 64-column K blocks per work item):
// pair tile 4 + 0.33 k, single tile 1.5 + 0.275 k.  The pair tile does four times the flops of the
// single one, so it wins whenever both variants have more than a wave of work; the single tile wins
// when a small step leaves most CTA pairs without a tile.
int hb_gemm_pick_step_variant(int map_variant, int rows, int N, int k_blocks, int k_splits, int num_sms) {
  if (map_variant != HB_GEMM_PAIR256 && map_variant != 128) return map_variant;
  if (rows <= 128) return 128;   // one row tile: the pair's second CTA would hold no rows
  const int ks = k_splits > 1 ? k_splits : 1;
  const double k = static_cast<double>((k_blocks + ks - 1) / ks);
  const long pairs = num_sms / 2 > 0 ? num_sms / 2 : 1;
  const long u_pair = static_cast<long>((rows + 255) / 256) * ((N + 255) / 256) * ks;
  const long u_single = static_cast<long>((rows + 127) / 128) * ((N + 127) / 128) * ks;
  const double t_pair = static_cast<double>((u_pair + pairs - 1) / pairs) * (4.0 + 0.33 * k);
  const double t_single = static_cast<double>((u_single + num_sms - 1) / num_sms) * (1.5 + 0.275 * k);
  return t_single * 1.05 < t_pair ? 128 : HB_GEMM_PAIR256;
}

int hb_gemm_box_rows(int variant) { return variant == HB_GEMM_PAIR256 ? 128 : variant; }

// Tile walk of a launch (see the kernel).  A's share of one work item, over all row tiles, is
// M x (K per item) x 2 bytes.  While that fits comfortably in L2 next to the B tiles of a wave, rows
// go fastest over the whole M and every B tile is read from DRAM once.  The 7B-class down projection
// is the launch where it does not (4096 x 7168 x 2 B = 59 MB per K half; each half of the L2 caches
// what its own SMs read, and every wave of 74 tile pairs touches all 16 row tiles): there the walk
// uses bands of row tiles whose share of A is about a quarter of L2, which makes a wave's footprint
// nearly square (8 row tiles x 9 column tiles).  Measured on that launch (profiler, DRAM read +
// write): 838 MB rows-fastest, 774 MB with bands of 8; the step time is the same within noise.
// Eviction hints on the loads (A evict-last, B evict-first) brought 755 MB but cost 0.7 ms per 7B
// step (three alternating runs), so the automatic choice leaves them off; they stay reachable
// through hb_gemm_set_walk.
static int g_band_override = -1;   // >= 0: test / tuning override of the band (0 = whole M)
static int g_hint_override = -1;
static int g_cta_limit = 0;        // > 0: launches use at most this many CTAs (an even number for CTA pairs)
void hb_gemm_walk_override(int band, int hints) { g_band_override = band; g_hint_override = hints; }
void hb_gemm_cta_limit(int max_ctas) { g_cta_limit = max_ctas; }

void hb_gemm_pick_walk(int variant, int epi, GemmArgs* g) {
  const int tile_rows = (variant == HB_GEMM_PAIR256) ? 256 : 128;
  const int ks = ((epi == HB_EPI_LORA_DOWN || epi == HB_EPI_RESID_F32) && g->k_splits > 1) ? g->k_splits : 1;
  const long k_item = (static_cast<long>(g->K) + ks - 1) / ks;
  const long a_tile_bytes = static_cast<long>(tile_rows) * k_item * 2;
  const int m_tiles = (g->M + tile_rows - 1) / tile_rows;
  g->raster_band = 0;
  g->l2_hints = 0;
  if (static_cast<long>(m_tiles) * a_tile_bytes > 40l * 1024 * 1024) {
    long band = (30l * 1024 * 1024) / a_tile_bytes;
    if (band < 1) band = 1;
    if (band < m_tiles) {
      g->raster_band = static_cast<int>(band);
      g->l2_hints = 0;
    }
  }
  if (g_band_override >= 0) g->raster_band = g_band_override;
  if (g_hint_override >= 0) g->l2_hints = g_hint_override;
}

int hb_gemm_launch(const CUtensorMap& tmA, const CUtensorMap& tmB, int variant, int epi, const GemmArgs& a,
                   int num_sms, cudaStream_t s, const CUtensorMap* tmA2, const CUtensorMap* tmB2, bool pdl) {
  if ((a.k2_blocks > 0) != (tmA2 != nullptr && tmB2 != nullptr) || a.k2_blocks < 0) return HB_ERR_BAD_ARG;
  if (epi == HB_EPI_LORA_DOWN && (a.k_splits < 1 || (a.k_splits > 1 && (!a.split_part || !a.split_counters))))
    return HB_ERR_BAD_ARG;
  if (epi == HB_EPI_RESID_F32 && a.k_splits > 1 && !a.split_counters) return HB_ERR_BAD_ARG;
  // without an extension the second pair is never read; pass the first so the parameters are valid maps
  const CUtensorMap& a2 = tmA2 ? *tmA2 : tmA;
  const CUtensorMap& b2 = tmB2 ? *tmB2 : tmB;
  GemmArgs g = a;
  hb_gemm_pick_walk(variant, epi, &g);
  if (g_cta_limit > 0 && g_cta_limit < num_sms) num_sms = g_cta_limit;
  if (variant == HB_GEMM_PAIR256) return launch_bn<256, 2>(tmA, tmB, a2, b2, epi, g, num_sms, s, pdl);
  if (variant == 256) return launch_bn<256, 1>(tmA, tmB, a2, b2, epi, g, num_sms, s, pdl);
  if (variant == 128) return launch_bn<128, 1>(tmA, tmB, a2, b2, epi, g, num_sms, s, pdl);
  return HB_ERR_BAD_ARG;
}
