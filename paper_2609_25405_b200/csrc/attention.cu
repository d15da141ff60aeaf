// Varlen causal attention over the paged KV cache for every row of the mixed batch
// (Section 3.2: decode tokens attend over their cached context, embedding / prefill chunks
// attend causally over their own earlier chunks plus themselves).  Row j of a segment has
// position pos = pos_start + j and sees keys 0 .. pos of its own request; all keys, the
// row's own included, are read from the pages (the append kernel ran before).
//
// Bring-up version: one warp per (row, query head), online softmax in fp32.
#include "hb_internal.h"

namespace {

template <int E>  // elements of the head dimension per lane: Dh = 32 * E
__global__ void __launch_bounds__(128)
attn_rowwarp_kernel(const __nv_bfloat16* __restrict__ q, KvGeom kv, int layer,
                    const int32_t* __restrict__ row_seg, const int32_t* __restrict__ row_pos,
                    const hb_seg* __restrict__ segs, const int32_t* __restrict__ pages,
                    __nv_bfloat16* __restrict__ out, int Hq, float scale, uint32_t* status) {
  const int t = blockIdx.x;
  const int head = blockIdx.y * 4 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (head >= Hq) return;
  const int Dh = kv.Dh;
  const int hk = head / (Hq / kv.Hkv);
  const int pos = row_pos[t];
  const hb_seg sg = segs[row_seg[t]];
  float qv[E];
  {
    const __nv_bfloat16* qp = q + (static_cast<size_t>(t) * Hq + head) * Dh + lane * E;
#pragma unroll
    for (int e = 0; e < E; ++e) qv[e] = __bfloat162float(qp[e]) * scale;
  }
  float m = -INFINITY, l = 0.0f, acc[E];
#pragma unroll
  for (int e = 0; e < E; ++e) acc[e] = 0.0f;
  const __nv_bfloat16* lbase = kv.arena + layer * kv.layer_stride;
  const int64_t head_stride = static_cast<int64_t>(kv.P) * Dh;
  for (int s = 0; s <= pos; ++s) {
    const int blk = s / kv.P, slot = s - blk * kv.P;
    const int page = pages[sg.pt_start + blk];
    if (page < 0 || page >= kv.n_pages) {
      if (lane == 0) atomicOr(status, HB_DEV_ATTN_BAD_INDEX);
      return;
    }
    const __nv_bfloat16* kp = lbase + page * kv.page_stride + hk * head_stride + slot * Dh + lane * E;
    const __nv_bfloat16* vp = kp + kv.Hkv * head_stride;
    float dot = 0.0f;
#pragma unroll
    for (int e = 0; e < E; ++e) dot += qv[e] * __bfloat162float(kp[e]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
    const float m_new = fmaxf(m, dot);
    const float corr = __expf(m - m_new);
    const float p = __expf(dot - m_new);
    l = l * corr + p;
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = acc[e] * corr + p * __bfloat162float(vp[e]);
    m = m_new;
  }
  const float inv = 1.0f / l;
  __nv_bfloat16* op = out + (static_cast<size_t>(t) * Hq + head) * Dh + lane * E;
#pragma unroll
  for (int e = 0; e < E; ++e) op[e] = __float2bfloat16(acc[e] * inv);
}

}  // namespace

int hb_launch_attention(hb_ctx* c, const KvGeom& kv, int layer, cudaStream_t s) {
  const int Hq = c->cfg.n_heads;
  const dim3 grid(c->dd.T, (Hq + 3) / 4);
  const float scale = 1.0f / sqrtf(static_cast<float>(c->cfg.head_dim));
  if (c->cfg.head_dim == 64)
    attn_rowwarp_kernel<2><<<grid, 128, 0, s>>>(c->q, kv, layer, c->dd.row_seg, c->dd.row_pos, c->dd.segs,
                                                 c->dd.pages, c->attn_out, Hq, scale, c->status);
  else if (c->cfg.head_dim == 128)
    attn_rowwarp_kernel<4><<<grid, 128, 0, s>>>(c->q, kv, layer, c->dd.row_seg, c->dd.row_pos, c->dd.segs,
                                                 c->dd.pages, c->attn_out, Hq, scale, c->status);
  else
    return HB_ERR_UNSUPPORTED;
  return cudaGetLastError() == cudaSuccess ? HB_OK : HB_ERR_CUDA;
}
