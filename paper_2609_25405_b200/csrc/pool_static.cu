// hb_pool_chunk_noalloc: the incremental pooler for callers that cannot allocate device memory.
//
// Every other compute entry point of this library needs an hb_ctx, and creating one allocates the
// workspace (or needs a caller-supplied one).  Some callers have neither option: a serving process
// whose own allocator took all device memory at start-up, or code called from a place where a
// device allocation would fail or stall the device.  For them this file keeps the pooler's
// scratch (per-block partial sums, the arrival counter, a status word) in a fixed array that is
// part of the loaded library image: every GPU that loads the library holds it (1 MiB + 256 B)
// until the process exits.  The price is a size limit and no concurrency: all calls on a device
// share the one array.
#include <mutex>

#include "hb_internal.h"
#include "pool_block.cuh"

namespace {

constexpr int MAX_ROWS = HB_NOALLOC_MAX_ROWS;       // rows of one chunk
constexpr int MAX_D = HB_NOALLOC_MAX_DMODEL;        // hidden size
constexpr int MAX_BLOCKS = MAX_ROWS / 32;           // one partial-sum record per block of 32 rows
constexpr size_t PART_FLOATS = static_cast<size_t>(MAX_BLOCKS) * MAX_D;
constexpr int TAIL_WORDS = 64;                      // [0] arrival counter, [1] status word

// Partial sums followed by the tail words.  In host code this name is only a handle for
// cudaGetSymbolAddress; it is not a device address.
static __device__ __align__(256) float g_pool_scratch[PART_FLOATS + TAIL_WORDS];

__global__ void __launch_bounds__(NORM_THREADS)
pool_chunk_static_kernel(float* __restrict__ scratch, const float* __restrict__ x,
                         const __nv_bfloat16* __restrict__ gain, int n_rows, int mode, int first_chunk, int is_final,
                         float* __restrict__ slot_sum, uint32_t* __restrict__ slot_meta, float* __restrict__ out_emb,
                         int d, float eps) {
  uint32_t* tail = reinterpret_cast<uint32_t*>(scratch + PART_FLOATS);
  hb_seg sg;
  sg.kind = HB_KIND_EMBED_CHUNK; sg.q_start = 0; sg.q_len = n_rows; sg.pos_start = first_chunk ? 0 : 1;
  sg.pt_start = 0; sg.pt_len = 0; sg.pool_slot = 0; sg.pool_mode = mode; sg.is_final = is_final;
  sg.logits_row = -1; sg.emb_row = 0; sg.reserved = 0;
  const PoolItem it = pool_chunk_item(mode, 0, n_rows, first_chunk != 0, is_final != 0, blockIdx.x, gridDim.x);
  pool_block(it, sg, x, gain, scratch, tail, slot_sum, slot_meta, out_emb, d, eps, 1, tail + 1);
}

constexpr int MAX_DEVICES = 64;
std::mutex g_setup_mutex;
float* g_scratch_addr[MAX_DEVICES] = {};

// Device address of the scratch array on the current device, looked up once per device.
int scratch_for_current_device(float** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return HB_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_pool_scratch) != cudaSuccess || !p) return HB_ERR_CUDA;
    g_scratch_addr[dev] = static_cast<float*>(p);
  }
  *out = g_scratch_addr[dev];
  return HB_OK;
}

}  // namespace

extern "C" int hb_pool_chunk_noalloc(const float* x, const void* gain, int32_t n_rows, int32_t d_model, float rms_eps,
                                     int32_t mode, int32_t first_chunk, int32_t is_final, float* slot_sum,
                                     uint32_t* slot_meta, float* out_emb, void* stream) {
  if (!x || !gain || !slot_sum || !slot_meta || n_rows < 1 || d_model < 4 || (d_model & 3)) return HB_ERR_BAD_ARG;
  if (mode < HB_POOL_MEAN || mode > HB_POOL_WMEAN) return HB_ERR_BAD_ARG;
  if (is_final && !out_emb) return HB_ERR_BAD_ARG;
  if (!(rms_eps >= 0.0f)) return HB_ERR_BAD_ARG;
  // The kernel moves rows, slot and output as 16-byte vectors and the gain as 8-byte ones.  A caller
  // that carves these out of its own arena (the caller this entry is for) can easily hand over a
  // view that starts mid-vector: refuse it here instead of faulting on the device.
  auto off = [](const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) != 0; };
  if (off(x, 16) || off(slot_sum, 16) || off(out_emb, 16) || off(gain, 8) || off(slot_meta, 4)) return HB_ERR_BAD_ARG;
  // beyond the fixed scratch: refuse, never truncate
  if (n_rows > MAX_ROWS || d_model > MAX_D) return HB_ERR_TOO_LARGE;
  float* scratch = nullptr;
  const int rc = scratch_for_current_device(&scratch);
  if (rc != HB_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // the array keeps whatever the previous call left: the arrival counter and the status word must start at zero
  if (cudaMemsetAsync(scratch + PART_FLOATS, 0, TAIL_WORDS * sizeof(float), s) != cudaSuccess) return HB_ERR_CUDA;
  const int blocks = (mode == HB_POOL_MEAN || mode == HB_POOL_WMEAN) ? (n_rows + 31) / 32 : 1;
  pool_chunk_static_kernel<<<blocks, NORM_THREADS, 0, s>>>(scratch, x, static_cast<const __nv_bfloat16*>(gain), n_rows,
                                                           mode, first_chunk != 0, is_final != 0, slot_sum, slot_meta,
                                                           out_emb, d_model, rms_eps);
  return cudaGetLastError() == cudaSuccess ? HB_OK : HB_ERR_CUDA;
}
