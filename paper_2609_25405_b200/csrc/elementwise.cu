// Memory-bound stages of the mixed step: token gather + RMSNorm, RMSNorm, final RMSNorm fused with the incremental pooler (Section 3.3, Eq. 1-2 and the
// last-token head) and with the hi/lo split that feeds the LM head, greedy argmax.
// All global accesses are 16-byte vectors; row statistics use warp shuffles; sums run in a
// fixed order (no floating-point atomics), so results do not depend on what else is batched.
#include "hb_internal.h"
#include "pool_block.cuh"
#include "ptx.cuh"

namespace {

// Activations leave these kernels as fp16 (three more mantissa bits than bf16); finite values
// saturate at the largest finite half, NaN stays NaN.
__device__ __forceinline__ float sat_h(float v) { return sat_half_range(v); }

__device__ __forceinline__ uint2 float4_to_f16x4(float4 v) {
  __half2 a = __floats2half2_rn(sat_h(v.x), sat_h(v.y)), b = __floats2half2_rn(sat_h(v.z), sat_h(v.w));
  uint2 r;
  r.x = *reinterpret_cast<uint32_t*>(&a);
  r.y = *reinterpret_cast<uint32_t*>(&b);
  return r;
}

__device__ __forceinline__ void f16x4_to_float4(uint2 raw, float4& o) {
  const float2 fa = __half22float2(*reinterpret_cast<const __half2*>(&raw.x));
  const float2 fb = __half22float2(*reinterpret_cast<const __half2*>(&raw.y));
  o = make_float4(fa.x, fa.y, fb.x, fb.y);
}

// x[t,:] = E[tok[t],:] (kept in fp32 as the residual stream); h[t,:] = fp16(rmsnorm(x) * gain).
// GATHER = false: x is read instead.  NV = 16-byte vectors a thread holds: 4 covers d_model <= 4096 in
// few enough registers for eight blocks per SM (more rows in flight per SM), 8 covers d_model <= 8192.
template <bool GATHER, int NV>
__global__ void __launch_bounds__(NORM_THREADS, NV == 4 ? 8 : 4)
norm_kernel(const int32_t* __restrict__ tok, const __nv_bfloat16* __restrict__ E,
            const __nv_bfloat16* __restrict__ gain, float* __restrict__ x, __half* __restrict__ h,
            int d, float eps, uint32_t* __restrict__ status) {
  grid_dep_wait();
  grid_dep_launch();
  __shared__ float red[32];
  const int t = blockIdx.x;
  const int nv = d >> 2;
  float4 buf[NV];
  float ss = 0.0f;
  float* xrow = x + static_cast<size_t>(t) * d;
  const __nv_bfloat16* erow = GATHER ? E + static_cast<size_t>(tok[t]) * d : nullptr;
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const int v = threadIdx.x + i * NORM_THREADS;
    if (v < nv) {
      if (GATHER) {
        bf16x4_to_float4(*reinterpret_cast<const uint2*>(erow + 4 * v), buf[i]);
        *reinterpret_cast<float4*>(xrow + 4 * v) = buf[i];
      } else {
        buf[i] = *reinterpret_cast<const float4*>(xrow + 4 * v);
      }
      ss += buf[i].x * buf[i].x + buf[i].y * buf[i].y + buf[i].z * buf[i].z + buf[i].w * buf[i].w;
    }
  }
  const float tot = block_sum(ss, red);
  const float rstd = rsqrtf(tot / static_cast<float>(d) + eps);
  __half* hrow = h + static_cast<size_t>(t) * d;
  bool range = false;
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const int v = threadIdx.x + i * NORM_THREADS;
    if (v < nv) {
      float4 g;
      bf16x4_to_float4(*reinterpret_cast<const uint2*>(gain + 4 * v), g);
      float4 o = make_float4(buf[i].x * rstd * g.x, buf[i].y * rstd * g.y, buf[i].z * rstd * g.z,
                             buf[i].w * rstd * g.w);
      range |= outside_half_range(o.x) | outside_half_range(o.y) | outside_half_range(o.z) | outside_half_range(o.w);
      *reinterpret_cast<uint2*>(hrow + 4 * v) = float4_to_f16x4(o);
    }
  }
  // a normed row that does not fit fp16 (a NaN in the residual stream, a gain far above 1) is reported
  if (range) atomicOr(status, HB_DEV_F16_RANGE);
}

// Final RMSNorm of the rows that feed the LM head, written as a (hi, lo) fp16 pair:
// hi = fp16(y), lo = fp16(y - hi), interleaved in blocks of 64 columns
// ([hi 0..63 | lo 0..63 | hi 64..127 | ...]).  The LM-head GEMM runs over 2d columns with each
// weight k-block used twice, which restores near-fp32 input precision for the logits.
__global__ void __launch_bounds__(NORM_THREADS)
final_logit_rows_kernel(const float* __restrict__ x, const __nv_bfloat16* __restrict__ gain,
                        const int32_t* __restrict__ logit_src, __half* __restrict__ out, int d, float eps) {
  grid_dep_wait();
  grid_dep_launch();
  __shared__ float red[32];
  const int i = blockIdx.x;
  const int t = logit_src[i];
  const int nv = d >> 2;
  const float* xrow = x + static_cast<size_t>(t) * d;
  float4 buf[MAX_VEC];
  float ss = 0.0f;
#pragma unroll
  for (int k = 0; k < MAX_VEC; ++k) {
    const int v = threadIdx.x + k * NORM_THREADS;
    if (v < nv) {
      buf[k] = *reinterpret_cast<const float4*>(xrow + 4 * v);
      ss += buf[k].x * buf[k].x + buf[k].y * buf[k].y + buf[k].z * buf[k].z + buf[k].w * buf[k].w;
    }
  }
  const float rstd = rsqrtf(block_sum(ss, red) / static_cast<float>(d) + eps);
  __half* orow = out + static_cast<size_t>(i) * 2 * d;
#pragma unroll
  for (int k = 0; k < MAX_VEC; ++k) {
    const int v = threadIdx.x + k * NORM_THREADS;
    if (v < nv) {
      float4 g;
      bf16x4_to_float4(*reinterpret_cast<const uint2*>(gain + 4 * v), g);
      const float4 y = make_float4(buf[k].x * rstd * g.x, buf[k].y * rstd * g.y, buf[k].z * rstd * g.z,
                                   buf[k].w * rstd * g.w);
      const uint2 hi = float4_to_f16x4(y);
      float4 hf;
      f16x4_to_float4(hi, hf);
      const uint2 lo = float4_to_f16x4(make_float4(y.x - hf.x, y.y - hf.y, y.z - hf.z, y.w - hf.w));
      const int c = 4 * v;
      __half* dst = orow + (c >> 6) * 128 + (c & 63);
      *reinterpret_cast<uint2*>(dst) = hi;
      *reinterpret_cast<uint2*>(dst + 64) = lo;
    }
  }
}

__global__ void __launch_bounds__(NORM_THREADS)
final_pool_kernel(const float* __restrict__ x, const __nv_bfloat16* __restrict__ gain,
                  const PoolItem* __restrict__ items, const hb_seg* __restrict__ segs, float* __restrict__ part,
                  uint32_t* __restrict__ counters, float* __restrict__ pool_sum, uint32_t* __restrict__ pool_meta,
                  float* __restrict__ out_emb, int d, float eps, int n_slots, uint32_t* status,
                  float* __restrict__ rowbuf, int rowbuf_rows) {
  grid_dep_wait();
  grid_dep_launch();
  const PoolItem it = items[blockIdx.x];
  const hb_seg sg = segs[it.seg];
  pool_block(it, sg, x, gain, part, counters, pool_sum, pool_meta, out_emb, d, eps, n_slots, status, rowbuf,
             rowbuf_rows);
}

// The pooler on its own: one chunk of one request, rows x[0 .. n_rows), slot 0 of a one-slot pool.
// Block b handles rows [32 b, 32 b + 32) (mean) or the last row (last-token head).
__global__ void __launch_bounds__(NORM_THREADS)
pool_chunk_kernel(const float* __restrict__ x, const __nv_bfloat16* __restrict__ gain, int n_rows, int mode,
                  int first_chunk, int is_final, float* __restrict__ part, uint32_t* __restrict__ counters,
                  float* __restrict__ slot_sum, uint32_t* __restrict__ slot_meta, float* __restrict__ out_emb, int d,
                  float eps, uint32_t* status) {
  hb_seg sg;
  sg.kind = HB_KIND_EMBED_CHUNK; sg.q_start = 0; sg.q_len = n_rows; sg.pos_start = first_chunk ? 0 : 1;
  sg.pt_start = 0; sg.pt_len = 0; sg.pool_slot = 0; sg.pool_mode = mode; sg.is_final = is_final;
  sg.logits_row = -1; sg.emb_row = 0; sg.reserved = 0;
  const PoolItem it = pool_chunk_item(mode, 0, n_rows, first_chunk != 0, is_final != 0, blockIdx.x, gridDim.x);
  pool_block(it, sg, x, gain, part, counters, slot_sum, slot_meta, out_emb, d, eps, 1, status);
}

__global__ void __launch_bounds__(256)
argmax_kernel(const float* __restrict__ logits, int V, int32_t* __restrict__ out) {
  __shared__ float bv[8];
  __shared__ int bi[8];
  const float* row = logits + static_cast<size_t>(blockIdx.x) * V;
  float best = -INFINITY;
  int idx = 0x7fffffff;
  for (int c = threadIdx.x; c < V; c += blockDim.x) {
    const float v = row[c];
    if (v > best || (v == best && c < idx)) { best = v; idx = c; }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, best, o);
    const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
    if (ov > best || (ov == best && oi < idx)) { best = ov; idx = oi; }
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) { bv[warp] = best; bi[warp] = idx; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < 8; ++w)
      if (bv[w] > best || (bv[w] == best && bi[w] < idx)) { best = bv[w]; idx = bi[w]; }
    out[blockIdx.x] = idx;
  }
}

// Weight repack: bf16 -> fp16, element by element (in place allowed: each thread reads its 8 values
// before it writes them).  Exact for 2^-14 <= |w| <= 65504; smaller magnitudes land on the fp16
// subnormal grid (absolute error <= 2^-25), larger ones saturate.
__global__ void __launch_bounds__(256)
bf16_to_f16_kernel(const __nv_bfloat16* src, __half* dst, size_t n_vec, size_t n) {
  const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
  for (size_t v = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; v < n_vec; v += stride) {
    const uint4 raw = *reinterpret_cast<const uint4*>(src + v * 8);
    float4 a, b;
    bf16x4_to_float4(make_uint2(raw.x, raw.y), a);
    bf16x4_to_float4(make_uint2(raw.z, raw.w), b);
    const uint2 lo = float4_to_f16x4(a), hi = float4_to_f16x4(b);
    *reinterpret_cast<uint4*>(dst + v * 8) = make_uint4(lo.x, lo.y, hi.x, hi.y);
  }
  if (blockIdx.x == 0 && threadIdx.x == 0)
    for (size_t i = n_vec * 8; i < n; ++i) dst[i] = __float2half_rn(sat_h(__bfloat162float(src[i])));
}

// Failure-path self-test: one thread waits, with the same bounded wait the pipelines use, on an
// mbarrier that nothing ever arrives on.  The wait gives up after `limit_ns`, the kernel raises a
// status bit and returns normally: no trap, no fault, the context stays usable.
__global__ void wait_expiry_selftest_kernel(uint64_t limit_ns, uint32_t* status) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    mbar_init_fence();
    if (!mbar_wait(smem_u32(&bar), 0u, nullptr, limit_ns)) atomicOr(status, HB_DEV_SELFTEST_WAIT_EXPIRED);
  }
}

int check_launch() { return cudaGetLastError() == cudaSuccess ? HB_OK : HB_ERR_CUDA; }

}  // namespace

int hb_launch_embed_norm(hb_ctx* c, const void* tok_emb, const void* gain, cudaStream_t s) {
  if (c->cfg.d_model <= 4 * 4 * NORM_THREADS)
    return hb_launch_kernel(norm_kernel<true, 4>, c->dd.T, NORM_THREADS, 0, s, c->pdl, c->dd.tok,
                            static_cast<const __nv_bfloat16*>(tok_emb), static_cast<const __nv_bfloat16*>(gain), c->x,
                            c->h, c->cfg.d_model, c->cfg.rms_eps, c->status);
  return hb_launch_kernel(norm_kernel<true, MAX_VEC>, c->dd.T, NORM_THREADS, 0, s, c->pdl, c->dd.tok,
                          static_cast<const __nv_bfloat16*>(tok_emb), static_cast<const __nv_bfloat16*>(gain), c->x,
                          c->h, c->cfg.d_model, c->cfg.rms_eps, c->status);
}

int hb_launch_rmsnorm(hb_ctx* c, const void* gain, cudaStream_t s) {
  if (c->cfg.d_model <= 4 * 4 * NORM_THREADS)
    return hb_launch_kernel(norm_kernel<false, 4>, c->dd.T, NORM_THREADS, 0, s, c->pdl, nullptr, nullptr,
                            static_cast<const __nv_bfloat16*>(gain), c->x, c->h, c->cfg.d_model, c->cfg.rms_eps,
                            c->status);
  return hb_launch_kernel(norm_kernel<false, MAX_VEC>, c->dd.T, NORM_THREADS, 0, s, c->pdl, nullptr, nullptr,
                          static_cast<const __nv_bfloat16*>(gain), c->x, c->h, c->cfg.d_model, c->cfg.rms_eps,
                          c->status);
}

int hb_launch_final(hb_ctx* c, const void* gain, float* pool_sum, uint32_t* pool_meta, int n_slots,
                    float* rowbuf, int rowbuf_rows, float* out_emb, cudaStream_t s) {
  const __nv_bfloat16* g = static_cast<const __nv_bfloat16*>(gain);
  if (c->dd.n_logit > 0) {
    if (hb_launch_kernel(final_logit_rows_kernel, c->dd.n_logit, NORM_THREADS, 0, s, c->pdl, c->x, g, c->dd.logit_src,
                         c->logit_in, c->cfg.d_model, c->cfg.rms_eps) != HB_OK)
      return HB_ERR_CUDA;
  }
  if (c->dd.n_pool_items > 0) {
    if (hb_launch_kernel(final_pool_kernel, c->dd.n_pool_items, NORM_THREADS, 0, s, c->pdl, c->x, g, c->dd.pool_items,
                         c->dd.segs, c->pool_part, c->counters, pool_sum, pool_meta, out_emb, c->cfg.d_model,
                         c->cfg.rms_eps, n_slots, c->status, rowbuf, rowbuf_rows) != HB_OK)
      return HB_ERR_CUDA;
  }
  return HB_OK;
}

int hb_launch_bf16_to_f16(const void* src, void* dst, size_t n, cudaStream_t s) {
  if (n == 0) return HB_OK;
  const size_t n_vec = n / 8;
  size_t blocks = (n_vec + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  if (blocks < 1) blocks = 1;
  bf16_to_f16_kernel<<<static_cast<unsigned>(blocks), 256, 0, s>>>(static_cast<const __nv_bfloat16*>(src),
                                                                   static_cast<__half*>(dst), n_vec, n);
  return check_launch();
}

int hb_launch_pool_chunk(hb_ctx* c, const float* x, const void* gain, int n_rows, int mode, int first_chunk,
                         int is_final, float* slot_sum, uint32_t* slot_meta, float* out_emb, cudaStream_t s) {
  const int blocks = (mode == HB_POOL_MEAN || mode == HB_POOL_WMEAN) ? (n_rows + 31) / 32 : 1;
  pool_chunk_kernel<<<blocks, NORM_THREADS, 0, s>>>(x, static_cast<const __nv_bfloat16*>(gain), n_rows, mode,
                                                    first_chunk, is_final, c->pool_part, c->counters, slot_sum,
                                                    slot_meta, out_emb, c->cfg.d_model, c->cfg.rms_eps, c->status);
  return check_launch();
}

int hb_launch_wait_expiry_selftest(hb_ctx* c, uint64_t limit_ns, cudaStream_t s) {
  wait_expiry_selftest_kernel<<<1, 32, 0, s>>>(limit_ns, c->status);
  return check_launch();
}

int hb_launch_argmax(const float* logits, int n_rows, int V, int32_t* out, cudaStream_t s) {
  if (n_rows <= 0) return HB_OK;
  argmax_kernel<<<n_rows, 256, 0, s>>>(logits, V, out);
  return check_launch();
}
