// coopt_paged_decode_static: paged decode for callers that cannot hand the library a
// workspace because they cannot allocate device memory at the point of the call -- an
// inference-runtime plug-in whose enqueue hook is forbidden to allocate, a serving loop that
// gave every free byte of the device to its own pool at start-up (so that a late cudaMalloc
// fails or stalls the whole device while it synchronises), or a plain C host program with no
// device allocator of its own.  The split-KV partials and the control words live in a
// fixed array inside the library image instead.  The paper has no counterpart of this call;
// it computes exactly what coopt_paged_decode computes.
#include <mutex>

#include "coopt_common.cuh"

namespace {

// Scratch of the static variant.  Every device that loads the library holds these bytes until
// the process exits.  All calls on a device share it.
static __device__ __align__(256) unsigned char g_static_scratch[COOPT_STATIC_SCRATCH_BYTES];

// Device address of the array on the current device.  In host code the symbol's name is only a
// handle; the address a kernel may use comes from the runtime, once per device.
int static_scratch_address(void** out) {
  static void* address[64] = {};
  static bool known[64] = {};
  static std::mutex mu;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return COOPT_ERR_CUDA;
  std::lock_guard<std::mutex> lock(mu);
  if (!known[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return COOPT_ERR_CUDA;
    address[dev] = p;
    known[dev] = true;
  }
  *out = address[dev];
  return COOPT_OK;
}

}  // namespace

extern "C" int coopt_paged_decode_static(const coopt_cache* cache, const void* q, void* out,
                                         const int32_t* block_table, int32_t max_blocks_per_seq,
                                         const int32_t* context_lens, int32_t batch, int32_t num_q_heads,
                                         float sm_scale, void* stream) {
  // every refusal comes before the first byte of the shared array is touched
  int rc = coopt::check_attention_args(cache, q, out, block_table, max_blocks_per_seq, context_lens, batch, num_q_heads);
  if (rc != COOPT_OK) return rc;
  if (batch == 0) return COOPT_OK;
  const size_t need = coopt_workspace_bytes(batch, num_q_heads, cache->num_kv_heads, cache->head_dim,
                                            max_blocks_per_seq, 0, batch);
  if (need == 0) return COOPT_ERR_INVALID_ARG;
  if (need > static_cast<size_t>(COOPT_STATIC_SCRATCH_BYTES)) return COOPT_ERR_WORKSPACE;   // beyond the built-in maximum
  void* scratch = nullptr;
  rc = static_scratch_address(&scratch);
  if (rc != COOPT_OK) return rc;
  // The array still holds whatever the previous call left: the control words must start at zero.
  rc = coopt_workspace_init(scratch, COOPT_STATIC_SCRATCH_BYTES, stream);
  if (rc != COOPT_OK) return rc;
  return coopt_paged_decode(cache, q, out, block_table, max_blocks_per_seq, context_lens, batch, num_q_heads,
                            sm_scale, scratch, COOPT_STATIC_SCRATCH_BYTES, stream);
}
