// The step's attention kernel: one launch per layer serves every row of the mixed batch (Section 3.2
// of the paper: decode tokens attend over their cached context, embedding / prefill chunks attend
// causally over their own earlier chunks plus themselves).  The host turns the batch descriptor
// into two cost-sorted item lists; a block of the grid takes one item:
//   chunk items of 65-128 query rows     -> tcgen05 body (attention_tc.cuh): tensor-bound
//   decode items, chunk items <= 64 rows -> mma.sync body (attention_dec.cuh): HBM-bound
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

// Block b -> (kind, item): the small items first, then the chunk tiles; both lists are sorted by
// cost, largest first, and blocks are dispatched roughly in index order.  The HBM-bound items
// stream while the machine is full of them and the tensor-bound tiles fill in as they drain; the
// other orders measured at the 7B configuration (chunk tiles first, or the two kinds alternating so
// that an SM tends to hold one of each) were 0.3 to 1 ms per step slower.
template <int DH, bool WITH_TC>
__global__ void __maxnreg__(160)
attn_varlen_kernel(const __grid_constant__ CUtensorMap kv_map, const hb_tc::TcParams tp, const hb_dec::AttnParams dp,
                   const int n_tc, const int n_small) {
  grid_dep_wait();
  grid_dep_launch();
  const int b = static_cast<int>(blockIdx.x);
  const bool chunk = b >= n_small;
  const int item = chunk ? b - n_small : b;
  if constexpr (WITH_TC) {
    if (chunk) { hb_tc::chunk_item<DH>(&kv_map, tp, item); return; }
    // A block of a kernel that can allocate tensor memory holds the SM's allocation permit until it
    // gives it up; a block that will never allocate does so at once, or no second block becomes
    // resident beside it (measured: one block per SM instead of two).
    if (threadIdx.x < 32) asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  hb_dec::small_item<DH>(&kv_map, dp, item);
}

template <int DH>
int launch(const CUtensorMap& kv_map, const hb_tc::TcParams& tp, const hb_dec::AttnParams& dp, int n_tc, int n_small,
           int max_pos, cudaStream_t s, bool pdl) {
  const int smem = std::max(n_tc > 0 ? hb_tc::smem_bytes<DH>() : 0, n_small > 0 ? hb_dec::smem_bytes<DH>(max_pos) : 0);
  static DynSmemState configured[2];   // per instantiation and per device
  if (smem > 227 * 1024) return HB_ERR_UNSUPPORTED;
  const int v = n_tc > 0 ? 1 : 0;
  auto kern = v ? attn_varlen_kernel<DH, true> : attn_varlen_kernel<DH, false>;
  if (hb_ensure_dyn_smem(reinterpret_cast<const void*>(kern), configured[v], smem) != HB_OK) return HB_ERR_CUDA;
  return hb_launch_kernel(kern, n_tc + n_small, ATTN_THREADS, smem, s, pdl, kv_map, tp, dp, n_tc, n_small);
}

}  // namespace

int hb_launch_attention(hb_ctx* c, const KvGeom& kv, const CUtensorMap& kv_map, int layer, cudaStream_t s, int which) {
  const int n_tc = (which & HB_ATTN_CHUNK_TILES) ? c->dd.n_tc_items : 0;
  const int n_small = (which & HB_ATTN_SMALL_ITEMS) ? c->dd.n_attn_items : 0;
  if (n_tc + n_small <= 0) return HB_OK;
  const hb_tc::TcParams tp = hb_tc::make_params(c, kv, layer);
  const hb_dec::AttnParams dp = hb_dec::make_params(c, kv, layer);
  if (c->cfg.head_dim == 64) return launch<64>(kv_map, tp, dp, n_tc, n_small, c->cfg.max_pos, s, c->pdl);
  if (c->cfg.head_dim == 128) return launch<128>(kv_map, tp, dp, n_tc, n_small, c->cfg.max_pos, s, c->pdl);
  return HB_ERR_UNSUPPORTED;
}
