// Dense decode attention for callers that cannot allocate device memory.
//
// Some hosts of this library have no way to hand it a workspace: a plugin that is given only the tensors
// of the operation it implements, code running inside a stream capture or under a memory pool that forbids
// cudaMalloc, a process whose device memory is fully committed to the KV cache.  ckv_dense_decode_static()
// serves them: it needs no context and no caller-provided scratch.  The split partials the attention kernel
// produces (and its last split merges) live in a fixed device array that is part of this library's
// image, so every GPU that loads the library holds CKV_STATIC_SCRATCH_BYTES of it until the process exits.
//
// Consequences the caller has to know:
//   * the array is shared by every call: two calls that overlap on the GPU (different streams, or the same
//     call from two host threads) race on it and produce garbage.  Serialise them;
//   * a problem whose partials do not fit returns CKV_ERR_CAPACITY before anything is launched;
//   * the first call on a device looks the array's device address up, and the first call with a given
//     (device, group size, kv_dtype) sets the attributes of the kernels that layout uses; make those first calls
//     outside any stream capture;
//   * problems only the device can see (a page id outside the pool) are skipped as everywhere else, but the
//     status word they are recorded in lives in the array and no call returns it: check page tables beforehand.
#include <mutex>

#include "ckv_internal.cuh"

#define CKV_STATIC_SCRATCH_BYTES (4u << 20)   // 4 MiB of split partials, followed by the words below
#define CKV_STATIC_TAIL_BYTES 1024            // 1 KiB: status word at +0, per-unit split counters at +256 (192 of them)

namespace {

// In host code these names are host-side stand-ins for the device arrays, not device addresses: the address a
// kernel may use comes from cudaGetSymbolAddress(), once per device.
static __device__ __align__(256) unsigned char g_static_scratch[CKV_STATIC_SCRATCH_BYTES + CKV_STATIC_TAIL_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void *g_scratch_ptr[kMaxDevices];   // device address of g_static_scratch on each device, null until looked up
int g_sm_count[kMaxDevices];
unsigned g_configured[kMaxDevices];  // bit (4 * kv_dtype + log2 G): the kernels of that layout have their attributes set

}  // namespace

extern "C" int ckv_dense_decode_static(const ckv_layout *layout, const void *q, const void *k_pool, const void *v_pool,
                                       const int32_t *page_table, const int32_t *seq_lens, int batch,
                                       int max_seq_len_host, void *out, float *lse, ckv_stream stream) {
  if (layout == nullptr || !q || !k_pool || !v_pool || !page_table || !seq_lens || !out) return CKV_ERR_INVALID_ARG;
  size_t stats_bytes = 0, work_bytes = 0;
  const int lst = ckv_query_sizes(layout, &stats_bytes, &work_bytes);   // host-only: validates the layout
  if (lst != CKV_OK) return lst;
  if (batch <= 0 || batch > layout->max_batch) return CKV_ERR_INVALID_ARG;
  if (max_seq_len_host <= 0 || (long long)max_seq_len_host > (long long)layout->max_blocks_per_seq * layout->block_size)
    return CKV_ERR_INVALID_ARG;

  // a context on the host stack: only the fields the dense path reads are filled in
  ckv_ctx c{};
  c.layout = *layout;
  if (c.layout.sm_scale == 0.f) c.layout.sm_scale = 1.0f / sqrtf((float)layout->head_dim);
  CkvDev &P = c.dev;
  P.Hq = layout->num_q_heads; P.Hkv = layout->num_kv_heads; P.G = P.Hq / P.Hkv;
  P.bs = layout->block_size; P.ppb = layout->block_size / layout->page_size;
  P.r = layout->var_groups; P.glayout = layout->group_layout;
  P.max_blocks = layout->max_blocks_per_seq; P.max_pages_per_seq = P.max_blocks * P.ppb;
  P.num_pages = layout->num_pages; P.sink = layout->sink_blocks; P.recent = layout->recent_blocks;
  P.scale = c.layout.sm_scale;
  P.row_elems = layout->stat_bf16 ? CKV_D : CKV_ROW_ELEMS;
  P.variant = layout->variant; P.half_var = 0.5f;   // the dense pass reads neither
  P.vhi = 0;
  P.scan_tile = layout->stat_bf16 ? CKV_SCAN_TILE_HS : CKV_SCAN_TILE;
  P.lg_bs = P.bs == 16 ? 4 : (P.bs == 32 ? 5 : 6);
  P.lg_tile = P.scan_tile == 32 ? 5 : 6;
  P.hkv_magic = (unsigned)((1ull << 32) / (unsigned)P.Hkv) + 1u;   // unused when Hkv == 1 (where it wraps)

  // the partials of the largest split count the launch heuristic may pick must fit the fixed array
  const size_t per_split = (size_t)batch * P.Hkv * P.G * CKV_PART_STRIDE * sizeof(float);
  if (per_split * CKV_MAX_SPLITS > CKV_STATIC_SCRATCH_BYTES) return CKV_ERR_CAPACITY;
  if ((size_t)batch * P.Hkv * sizeof(int) > CKV_STATIC_TAIL_BYTES - 256) return CKV_ERR_CAPACITY;

  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return ckv_record_cuda_error(e);
  if (dev < 0 || dev >= kMaxDevices) return ckv_record_cuda_error(cudaErrorInvalidDevice);
  {
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_scratch_ptr[dev] == nullptr) {   // once per device, with that device current
      void *ptr = nullptr;
      e = cudaGetSymbolAddress(&ptr, g_static_scratch);
      if (e == cudaSuccess) e = cudaDeviceGetAttribute(&g_sm_count[dev], cudaDevAttrMultiProcessorCount, dev);
      if (e != cudaSuccess) return ckv_record_cuda_error(e);
      if (ptr == nullptr) return ckv_record_cuda_error(cudaErrorInvalidSymbol);
      g_scratch_ptr[dev] = ptr;
    }
    // the attention kernels of this layout (one instantiation per group size and page type) opt in to their
    // shared memory once per device: a later call with another layout must not find the opt-in missing
    const int lg = P.G == 1 ? 0 : (P.G == 2 ? 1 : (P.G == 4 ? 2 : 3));
    const unsigned bit = 1u << (4 * (layout->kv_dtype == CKV_BF16 ? 0 : 1) + lg);
    if ((g_configured[dev] & bit) == 0) {
      e = ckv_configure_attn(&c);
      if (e == cudaSuccess) e = ckv_configure_attn_mma(&c);
      if (e != cudaSuccess) return ckv_record_cuda_error(e);
      g_configured[dev] |= bit;
    }
  }
  unsigned char *scratch = (unsigned char *)g_scratch_ptr[dev];
  P.attn_part = (float *)scratch;
  P.status = (int *)(scratch + CKV_STATIC_SCRATCH_BYTES);
  P.unit_done = (int *)(scratch + CKV_STATIC_SCRATCH_BYTES + 256);
  c.sm_count = g_sm_count[dev];

  cudaStream_t s = (cudaStream_t)stream;
  // the array keeps whatever the previous call left: the status word and the split counters must start at zero
  // (an interrupted call may have left counters behind); every partial that is read is rewritten by this call
  e = cudaMemsetAsync(P.status, 0, CKV_STATIC_TAIL_BYTES, s);
  if (e != cudaSuccess) return ckv_record_cuda_error(e);
  int n_splits = 0;
  bool merged = false;
  e = ckv_launch_attn(&c, true, q, k_pool, v_pool, page_table, seq_lens, nullptr, nullptr, 0, batch, max_seq_len_host,
                      0, out, lse, &n_splits, &merged, s);
  if (e != cudaSuccess) return ckv_record_cuda_error(e);
  if (!merged) {   // fp32 pages: the merge is a launch of its own
    e = ckv_launch_merge(&c, true, seq_lens, nullptr, n_splits, 0, batch, out, lse, s);
    if (e != cudaSuccess) return ckv_record_cuda_error(e);
  }
  return CKV_OK;
}
