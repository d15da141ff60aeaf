// Device code of the incremental pooler (Section 3.3 of the paper, Eq. 1-2 and the last-token head)
// and the small reduction helpers it shares with the other memory-bound kernels.  Included by the
// translation units that launch it.
#pragma once

#include "hb_internal.h"

namespace {

constexpr int NORM_THREADS = 256;
constexpr int MAX_VEC = 8;  // float4 per thread held in registers: d_model <= 256 * 4 * 8 = 8192

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Sum over the block; every thread gets the result.  red must hold 32 floats.
__device__ __forceinline__ float block_sum(float v, float* red) {
  v = warp_sum(v);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  __syncthreads();
  if (lane == 0) red[warp] = v;
  __syncthreads();
  float t = (lane < (blockDim.x >> 5)) ? red[lane] : 0.0f;
  t = warp_sum(t);
  return t;
}

__device__ __forceinline__ void bf16x4_to_float4(uint2 raw, float4& o) {
  const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&raw.x);
  const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162*>(&raw.y);
  const float2 fa = __bfloat1622float2(a), fb = __bfloat1622float2(b);
  o = make_float4(fa.x, fa.y, fb.x, fb.y);
}

// Work item of the pooler for block `block` of `n_blocks` of one chunk.  Additive heads (mean,
// weighted mean) take 32 rows per block; positional heads read one row (CLS: the first row of the
// first chunk, last-token: the last row of the final chunk) or none.
__device__ __forceinline__ PoolItem pool_chunk_item(int mode, int q_start, int n_rows, bool first_chunk, bool is_final,
                                                    int block, int n_blocks) {
  PoolItem it;
  it.seg = 0; it.block = block; it.n_blocks = n_blocks; it.part_base = 0; it.pad[0] = it.pad[1] = 0;
  if (mode == HB_POOL_MEAN || mode == HB_POOL_WMEAN || mode == HB_POOL_MAX) {
    it.row0 = q_start + block * 32;
    it.n_rows = min(32, n_rows - block * 32);
  } else if (mode == HB_POOL_CLS) {
    it.row0 = q_start;
    it.n_rows = first_chunk ? 1 : 0;
  } else {
    it.row0 = q_start + n_rows - 1;
    it.n_rows = is_final ? 1 : 0;
  }
  return it;
}

// Buffered head (Section 3.3): a head that needs every row at once keeps A(k) = [A(k-1); H(k)], the
// final hidden states of all rows seen so far, at O(n d) memory, and runs after the final chunk.
// The head built in is the element-wise maximum over the n rows.  Every chunk appends its rows
// (final RMSNorm applied, fp32) to the slot's row buffer at the rows' positions.  On the final chunk
// the head runs over all n rows: block b of the chunk's n_blocks takes its own 32 rows straight from
// the residual stream plus an equal share of the pos_start rows buffered by earlier steps, writes a
// partial maximum, and the block that arrives last combines the partials, L2-normalises and emits.
// The maximum is exact in any order, so the result does not depend on how the rows are shared out.
__device__ __forceinline__ void pool_block_buffered(const PoolItem& it, const hb_seg& sg, const float* __restrict__ x,
                                                    const __nv_bfloat16* __restrict__ gain, float* __restrict__ part,
                                                    uint32_t* __restrict__ counters, uint32_t* __restrict__ meta,
                                                    float* __restrict__ rowbuf, int rowbuf_rows,
                                                    float* __restrict__ out_emb, int d, float eps, uint32_t* status) {
  __shared__ float red_b[32];
  __shared__ float rstd_b[32];
  __shared__ uint32_t is_last_b;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nv = d >> 2;
  if (rowbuf == nullptr || sg.pos_start + sg.q_len > rowbuf_rows) {
    if (threadIdx.x == 0) atomicOr(status, HB_DEV_POOL_BAD_INDEX);
    return;
  }
  const bool first_chunk = (sg.pos_start == 0);
  const bool emit = (sg.is_final != 0);
  float* A = rowbuf + static_cast<size_t>(sg.pool_slot) * rowbuf_rows * d;
  for (int r = warp; r < it.n_rows; r += NORM_THREADS / 32) {
    const float* xrow = x + static_cast<size_t>(it.row0 + r) * d;
    float ss = 0.0f;
    for (int v = lane; v < nv; v += 32) {
      const float4 a = *reinterpret_cast<const float4*>(xrow + 4 * v);
      ss += a.x * a.x + a.y * a.y + a.z * a.z + a.w * a.w;
    }
    ss = warp_sum(ss);
    if (lane == 0) rstd_b[r] = rsqrtf(ss / static_cast<float>(d) + eps);
  }
  __syncthreads();
  // rows buffered by earlier steps that this block folds into its partial (final chunk only)
  const int share = (sg.pos_start + it.n_blocks - 1) / it.n_blocks;
  const int p0 = emit ? min(it.block * share, sg.pos_start) : 0;
  const int p1 = emit ? min(p0 + share, sg.pos_start) : 0;
  const int pos0 = sg.pos_start + (it.row0 - sg.q_start);     // position of the item's first row
  float* my_part = part + static_cast<size_t>(it.part_base + it.block) * d;
#pragma unroll 1
  for (int v = threadIdx.x; v < nv; v += NORM_THREADS) {
    float4 g;
    bf16x4_to_float4(*reinterpret_cast<const uint2*>(gain + 4 * v), g);
    float4 m = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
    for (int r = 0; r < it.n_rows; ++r) {
      const float4 a = *reinterpret_cast<const float4*>(x + static_cast<size_t>(it.row0 + r) * d + 4 * v);
      const float s = rstd_b[r];
      const float4 hv = make_float4(a.x * s * g.x, a.y * s * g.y, a.z * s * g.z, a.w * s * g.w);
      *reinterpret_cast<float4*>(A + static_cast<size_t>(pos0 + r) * d + 4 * v) = hv;
      m.x = fmaxf(m.x, hv.x); m.y = fmaxf(m.y, hv.y); m.z = fmaxf(m.z, hv.z); m.w = fmaxf(m.w, hv.w);
    }
    for (int pr = p0; pr < p1; ++pr) {
      const float4 hv = *reinterpret_cast<const float4*>(A + static_cast<size_t>(pr) * d + 4 * v);
      m.x = fmaxf(m.x, hv.x); m.y = fmaxf(m.y, hv.y); m.z = fmaxf(m.z, hv.z); m.w = fmaxf(m.w, hv.w);
    }
    if (emit) *reinterpret_cast<float4*>(my_part + 4 * v) = m;
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const uint32_t prev = atomicAdd(counters + it.seg, 1u);
    is_last_b = (prev + 1u == static_cast<uint32_t>(it.n_blocks)) ? 1u : 0u;
  }
  __syncthreads();
  if (!is_last_b) return;
  __threadfence();
  const uint32_t old_count = first_chunk ? 0u : meta[0];
  const uint32_t old_chunks = first_chunk ? 0u : meta[1];
  if (emit) {
    float4 e[MAX_VEC];
    float nrm = 0.0f;
#pragma unroll
    for (int k = 0; k < MAX_VEC; ++k) {
      const int v = threadIdx.x + k * NORM_THREADS;
      e[k] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (v < nv) {
        float4 m = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
        for (int b = 0; b < it.n_blocks; ++b) {
          const float4 q = __ldcg(reinterpret_cast<const float4*>(part + static_cast<size_t>(it.part_base + b) * d + 4 * v));
          m.x = fmaxf(m.x, q.x); m.y = fmaxf(m.y, q.y); m.z = fmaxf(m.z, q.z); m.w = fmaxf(m.w, q.w);
        }
        e[k] = m;
        nrm += m.x * m.x + m.y * m.y + m.z * m.z + m.w * m.w;
      }
    }
    const float tot = block_sum(nrm, red_b);
    const float inv = 1.0f / fmaxf(sqrtf(tot), 1e-12f);
    float* o = out_emb + static_cast<size_t>(sg.emb_row) * d;
#pragma unroll
    for (int k = 0; k < MAX_VEC; ++k) {
      const int v = threadIdx.x + k * NORM_THREADS;
      if (v < nv)
        *reinterpret_cast<float4*>(o + 4 * v) = make_float4(e[k].x * inv, e[k].y * inv, e[k].z * inv, e[k].w * inv);
    }
  }
  if (threadIdx.x == 0) {
    meta[0] = old_count + static_cast<uint32_t>(sg.q_len);
    meta[1] = old_chunks + 1u;
    meta[2] = static_cast<uint32_t>(sg.pool_mode);
    meta[3] = emit ? 1u : 0u;
    counters[it.seg] = 0u;
  }
}

// Final RMSNorm fused with the incremental pooler (Section 3.3).  One block per work item = a block
// of rows of one embedding segment.  Phase 1: one warp per row, shuffle-reduced sum of squares.
// Phase 2: each thread owns column vectors and adds w_j * x_j * rstd_j over the item's rows in row
// order.  The block's partial sum goes to scratch; the block that arrives last for a segment adds
// the partials in block order, applies the gain, and updates the slot:
//   S <- S + sum_j w_j H_j,  W <- W + sum_j w_j                       (Eq. 1-2)
// with w = 1 (mean) or w = position + 1 (weighted mean; W is then count (count + 1) / 2, so the
// integer token count is the only counter kept).  A request's first chunk overwrites the slot
// (S(0) = 0, W(0) = 0).  Positional heads keep one row: CLS stores the first row of the first chunk
// in S, last-token reads the last row of the final chunk.  On the final chunk the block emits
// S / W (or the retained row), L2-normalised.
__device__ __forceinline__ void pool_block(const PoolItem& it, const hb_seg& sg, const float* __restrict__ x,
                                           const __nv_bfloat16* __restrict__ gain, float* __restrict__ part,
                                           uint32_t* __restrict__ counters, float* __restrict__ pool_sum,
                                           uint32_t* __restrict__ pool_meta, float* __restrict__ out_emb, int d,
                                           float eps, int n_slots, uint32_t* status, float* __restrict__ rowbuf = nullptr,
                                           int rowbuf_rows = 0) {
  __shared__ float red[32];
  __shared__ float rstd_s[32];
  __shared__ uint32_t is_last_s;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nv = d >> 2;
  if (sg.pool_slot < 0 || sg.pool_slot >= n_slots) {
    if (threadIdx.x == 0) atomicOr(status, HB_DEV_POOL_BAD_INDEX);
    return;
  }
  if (sg.pool_mode == HB_POOL_MAX) {
    pool_block_buffered(it, sg, x, gain, part, counters, pool_meta + static_cast<size_t>(sg.pool_slot) * 4, rowbuf,
                        rowbuf_rows, out_emb, d, eps, status);
    return;
  }
  const bool first_chunk = (sg.pos_start == 0);
  const bool additive = (sg.pool_mode == HB_POOL_MEAN || sg.pool_mode == HB_POOL_WMEAN);
  const bool cls = (sg.pool_mode == HB_POOL_CLS);
  float* S = pool_sum + static_cast<size_t>(sg.pool_slot) * d;
  uint32_t* meta = pool_meta + static_cast<size_t>(sg.pool_slot) * 4;
  // tokens pooled before this chunk = position of the chunk's first row (only the last block writes meta)
  const uint32_t old_count = first_chunk ? 0u : meta[0];
  // phase 1: row statistics (item rows <= 32), with the row's weight folded in
  for (int r = warp; r < it.n_rows; r += NORM_THREADS / 32) {
    const float* xrow = x + static_cast<size_t>(it.row0 + r) * d;
    float ss = 0.0f;
    for (int v = lane; v < nv; v += 32) {
      const float4 a = *reinterpret_cast<const float4*>(xrow + 4 * v);
      ss += a.x * a.x + a.y * a.y + a.z * a.z + a.w * a.w;
    }
    ss = warp_sum(ss);
    if (lane == 0) {
      const float w = (sg.pool_mode == HB_POOL_WMEAN)
                          ? static_cast<float>(old_count + static_cast<uint32_t>(it.row0 + r - sg.q_start) + 1u)
                          : 1.0f;
      rstd_s[r] = rsqrtf(ss / static_cast<float>(d) + eps) * w;
    }
  }
  __syncthreads();
  // phase 2: column sums over the item's rows, fixed row order
  float* my_part = part + static_cast<size_t>(it.part_base + it.block) * d;
#pragma unroll 1
  for (int v = threadIdx.x; v < nv; v += NORM_THREADS) {
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int r = 0; r < it.n_rows; ++r) {
      const float4 a = *reinterpret_cast<const float4*>(x + static_cast<size_t>(it.row0 + r) * d + 4 * v);
      const float s = rstd_s[r];
      acc.x += a.x * s; acc.y += a.y * s; acc.z += a.z * s; acc.w += a.w * s;
    }
    *reinterpret_cast<float4*>(my_part + 4 * v) = acc;
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const uint32_t prev = atomicAdd(counters + it.seg, 1u);
    is_last_s = (prev + 1u == static_cast<uint32_t>(it.n_blocks)) ? 1u : 0u;
  }
  __syncthreads();
  if (!is_last_s) return;
  __threadfence();
  // segment tail: combine partials in block order, update the slot, maybe emit
  const uint32_t old_chunks = first_chunk ? 0u : meta[1];
  const uint32_t new_count = old_count + static_cast<uint32_t>(sg.q_len);
  const bool emit = (sg.is_final != 0);
  const bool from_rows = additive || (cls && first_chunk) || (sg.pool_mode == HB_POOL_LAST && emit);
  // total weight W: count for the mean, count (count + 1) / 2 for position weights
  const double W = (sg.pool_mode == HB_POOL_WMEAN) ? 0.5 * static_cast<double>(new_count) * (new_count + 1.0)
                                                   : static_cast<double>(new_count);
  const float inv_W = static_cast<float>(1.0 / W);
  float4 e[MAX_VEC];
  float nrm = 0.0f;
#pragma unroll
  for (int k = 0; k < MAX_VEC; ++k) {
    const int v = threadIdx.x + k * NORM_THREADS;
    e[k] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (v < nv && (from_rows || emit)) {
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      if (from_rows) {
        for (int b = 0; b < it.n_blocks; ++b) {
          const float4 p = __ldcg(reinterpret_cast<const float4*>(part + static_cast<size_t>(it.part_base + b) * d + 4 * v));
          acc.x += p.x; acc.y += p.y; acc.z += p.z; acc.w += p.w;
        }
        float4 g;
        bf16x4_to_float4(*reinterpret_cast<const uint2*>(gain + 4 * v), g);
        acc.x *= g.x; acc.y *= g.y; acc.z *= g.z; acc.w *= g.w;
      }
      if (additive) {
        if (!first_chunk) {
          const float4 o = *reinterpret_cast<const float4*>(S + 4 * v);
          acc.x += o.x; acc.y += o.y; acc.z += o.z; acc.w += o.w;
        }
        *reinterpret_cast<float4*>(S + 4 * v) = acc;
        acc.x *= inv_W; acc.y *= inv_W; acc.z *= inv_W; acc.w *= inv_W;
      } else if (cls) {
        if (first_chunk) *reinterpret_cast<float4*>(S + 4 * v) = acc;      // retain H_1 of the first chunk
        else acc = *reinterpret_cast<const float4*>(S + 4 * v);
      }
      e[k] = acc;
      nrm += acc.x * acc.x + acc.y * acc.y + acc.z * acc.z + acc.w * acc.w;
    }
  }
  if (emit) {
    const float tot = block_sum(nrm, red);
    const float inv = 1.0f / fmaxf(sqrtf(tot), 1e-12f);
    float* o = out_emb + static_cast<size_t>(sg.emb_row) * d;
#pragma unroll
    for (int k = 0; k < MAX_VEC; ++k) {
      const int v = threadIdx.x + k * NORM_THREADS;
      if (v < nv)
        *reinterpret_cast<float4*>(o + 4 * v) = make_float4(e[k].x * inv, e[k].y * inv, e[k].z * inv, e[k].w * inv);
    }
  }
  if (threadIdx.x == 0) {
    meta[0] = new_count;
    meta[1] = old_chunks + 1u;
    meta[2] = static_cast<uint32_t>(sg.pool_mode);
    meta[3] = emit ? 1u : 0u;
    counters[it.seg] = 0u;  // ready for the next step
  }
}

}  // namespace
