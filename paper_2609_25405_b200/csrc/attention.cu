// The step's attention kernel: one launch per layer serves every row of the mixed batch (Section 3.2
// of the paper: decode tokens attend over their cached context, embedding / prefill chunks attend
// causally over their own earlier chunks plus themselves).  The host turns the batch descriptor
// into two cost-sorted item lists; the blocks of the grid stay resident and take one item after the
// other:
//   chunk tiles of up to 128 query rows -> tcgen05 body (attention_tc.cuh): tensor-bound
//   decode items (one split of a row)   -> mma.sync body (attention_dec.cuh): HBM-bound
// Both bodies run with the same block size and register budget (two blocks per SM); shared memory
// is the larger of their needs.  A launch without chunk tiles runs an instantiation without the
// tcgen05 body.
#include "attention_dec.cuh"
#include "attention_tc.cuh"
#include "hb_internal.h"
#include "ptx.cuh"

namespace {

static_assert(hb_tc::TC_THREADS == hb_dec::ATT_THREADS, "one block size for both kinds of item");
constexpr int ATTN_THREADS = hb_tc::TC_THREADS;

// The blocks stay resident (two per SM) and take items one after the other: item b first for block
// b, then whatever an atomic ticket hands out, in list order: the small items first, then the chunk
// tiles; both lists are sorted by cost, largest first.  The HBM-bound items stream while the machine
// is full of them and the tensor-bound tiles fill in as they drain.  (One block per item left SM
// slots idle: with shared memory and registers nearly full, an SM admitted a new block only when the
// OLDER of its two resident blocks left, so the slot of a short item next to a long one stayed empty
// until the long one was done; measured on the chunk tiles of the 7B configuration: 242 of 296 slots
// busy on average.)
//
// queue[0] = tickets handed out, queue[1] = blocks that have left; the last block to leave zeroes
// both for the next launch.  The launches of one stream follow each other (each starts its work
// after the previous grid has completed), so one queue serves them all.
template <int DH, bool WITH_TC>
__global__ void __maxnreg__(160)
attn_varlen_kernel(const __grid_constant__ CUtensorMap kv_map, const hb_tc::TcParams tp, const hb_dec::AttnParams dp,
                   const int n_tc, const int n_small, uint32_t* const queue, const int smem_total) {
  grid_dep_wait();
  grid_dep_launch();
  extern __shared__ uint8_t smem_raw[];
  // the last 16 bytes of the window belong to the loop: [0] next item, [1] tensor-memory base, [2] ticket
  volatile uint32_t* slot = reinterpret_cast<volatile uint32_t*>(smem_raw + smem_total - 16);
  const uint32_t smem_base = smem_u32(smem_raw);
  const int tid = static_cast<int>(threadIdx.x);
  uint32_t tmem = 0;
  if constexpr (WITH_TC) {
    // one allocation for the block's lifetime; the permit is given up at once (a resident block that
    // still holds it keeps a second block from becoming resident)
    if (tid < 32) {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(const_cast<uint32_t*>(slot + 1))),
                   "r"(static_cast<uint32_t>(hb_tc::TcCfg<DH>::TMEM_COLS)) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    tmem = slot[1];
  }
  const uint32_t total = static_cast<uint32_t>(n_tc + n_small);
  constexpr uint32_t NONE = 0xfffffffeu, STOP = 0xffffffffu;
  // The ticket for the block's next item is taken by a thread that can wait for it without holding
  // anyone up.  A chunk tile (long: up to 64 key tiles): its TMA thread, when it has requested the last
  // key tile: late enough that items are handed out in the order blocks really finish (largest first
  // only pays off then), early enough that the atomic's latency hides behind the last tiles.  A small
  // item (short; its threads meet at a block barrier per key tile): the idle sixth warp, first thing,
  // behind the item's first loads.
  auto take_ticket = [&]() { slot[2] = atomicAdd(queue, 1u) + gridDim.x; };
  uint32_t b = blockIdx.x;
  while (b < total) {
    bool ok, live = true;
    const bool chunk = WITH_TC && b >= static_cast<uint32_t>(n_small);
    if (tid == (chunk ? 0 : hb_dec::ATT_COMPUTE + 32)) slot[2] = NONE;   // the thread that takes the ticket
    if constexpr (WITH_TC) {
      if (chunk) ok = hb_tc::chunk_item<DH>(&kv_map, tp, static_cast<int>(b) - n_small, tmem, &live, take_ticket);
      else ok = hb_dec::small_item<DH>(&kv_map, dp, static_cast<int>(b), take_ticket);
    } else {
      ok = hb_dec::small_item<DH>(&kv_map, dp, static_cast<int>(b), take_ticket);
    }
    fence_async_smem();   // this item's generic accesses to shared memory, before the next item's copies
    __syncthreads();
    if (tid == 0) {
      if constexpr (WITH_TC) {
        if (chunk) { if (live) hb_tc::retire_barriers<DH>(smem_base); }
        else hb_dec::retire_barriers<DH>(smem_base);
      } else {
        hb_dec::retire_barriers<DH>(smem_base);
      }
      uint32_t nxt = slot[2];
      if (nxt == NONE) nxt = atomicAdd(queue, 1u) + gridDim.x;   // an item that ended early
      slot[0] = ok ? nxt : STOP;
    }
    __syncthreads();
    b = slot[0];
  }
  if constexpr (WITH_TC) {
    tc_fence_before();
    __syncthreads();
    if (tid < 32) {
      tc_fence_after();
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem),
                   "r"(static_cast<uint32_t>(hb_tc::TcCfg<DH>::TMEM_COLS)) : "memory");
    }
  }
  if (tid == 0) {
    __threadfence();
    if (atomicAdd(queue + 1, 1u) == gridDim.x - 1u) {
      queue[0] = 0u;
      queue[1] = 0u;
    }
  }
}

int g_block_limit = 0;   // > 0: launches use at most this many blocks

template <int DH>
int launch(const CUtensorMap& kv_map, const hb_tc::TcParams& tp, const hb_dec::AttnParams& dp, int n_tc, int n_small,
           int max_pos, int num_sms, uint32_t* queue, cudaStream_t s, bool pdl) {
  const int smem = std::max(n_tc > 0 ? hb_tc::smem_bytes<DH>() : 0, n_small > 0 ? hb_dec::smem_bytes<DH>(max_pos) : 0) + 16;
  static DynSmemState configured[2];   // per instantiation and per device
  if (smem > 227 * 1024) return HB_ERR_UNSUPPORTED;
  const int v = n_tc > 0 ? 1 : 0;
  auto kern = v ? attn_varlen_kernel<DH, true> : attn_varlen_kernel<DH, false>;
  if (hb_ensure_dyn_smem(reinterpret_cast<const void*>(kern), configured[v], smem) != HB_OK) return HB_ERR_CUDA;
  int blocks = std::min(n_tc + n_small, 2 * num_sms);
  if (g_block_limit > 0) blocks = std::min(blocks, g_block_limit);
  return hb_launch_kernel(kern, blocks, ATTN_THREADS, smem, s, pdl, kv_map, tp, dp, n_tc, n_small, queue, smem);
}

}  // namespace

void hb_attn_block_limit(int max_blocks) { g_block_limit = max_blocks; }

int hb_launch_attention(hb_ctx* c, const KvGeom& kv, const CUtensorMap& kv_map, int layer, cudaStream_t s, int which) {
  const int n_tc = (which & HB_ATTN_CHUNK_TILES) ? c->dd.n_tc_items : 0;
  const int n_small = (which & HB_ATTN_SMALL_ITEMS) ? c->dd.n_attn_items : 0;
  if (n_tc + n_small <= 0) return HB_OK;
  const hb_tc::TcParams tp = hb_tc::make_params(c, kv, layer);
  const hb_dec::AttnParams dp = hb_dec::make_params(c, kv, layer);
  uint32_t* queue = c->status + HB_STATUS_ATTN_QUEUE_WORD;
  if (c->cfg.head_dim == 64) return launch<64>(kv_map, tp, dp, n_tc, n_small, c->cfg.max_pos, c->num_sms, queue, s, c->pdl);
  if (c->cfg.head_dim == 128) return launch<128>(kv_map, tp, dp, n_tc, n_small, c->cfg.max_pos, c->num_sms, queue, s, c->pdl);
  return HB_ERR_UNSUPPORTED;
}
