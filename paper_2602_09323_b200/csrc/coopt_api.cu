// Host side of the C ABI: argument checks, workspace arithmetic, dispatch to the launchers.
#include <mutex>
#include <utility>
#include <vector>

#include "coopt_common.cuh"

namespace coopt {

int launch_kv_write(const coopt_cache* c, const void* k, const void* v, int64_t stride, const int64_t* slots,
                    int num_tokens, cudaStream_t stream);
int launch_paged_decode(const coopt_cache* c, const void* q, void* out, const int32_t* block_table,
                        int32_t max_blocks_per_seq, const int32_t* context_lens, int32_t batch, int32_t num_q_heads,
                        float sm_scale, int32_t chunk_size, const int32_t* cu_q_lens, void* workspace, int planned_ctas,
                        cudaStream_t stream);
int launch_paged_prefill(const coopt_cache* c, const void* q, void* out, const int32_t* cu_q_lens,
                         const int32_t* block_table, int32_t max_blocks_per_seq, const int32_t* context_lens,
                         int32_t batch, int32_t num_q_heads, int32_t total_q, int32_t causal, float sm_scale,
                         void* workspace, cudaStream_t stream);
size_t decode_workspace_bytes(int planned_ctas, int group, int head_dim, int batch, int num_q_heads, int num_kv_heads,
                              int max_blocks_per_seq, int chunk_blocks, int max_chunks);
size_t plan_bytes(int planned_ctas, int batch, int num_kv_heads, int max_blocks_per_seq, int chunk_blocks);
int launch_decode_plan(const int32_t* block_table, int32_t max_blocks_per_seq, const int32_t* context_lens, int32_t batch,
                       int32_t num_kv_heads, int32_t num_blocks, int32_t chunk_size, int planned_ctas, void* plan,
                       cudaStream_t stream);
int launch_decode_planned(const coopt_cache* c, const void* plan, const void* k_new, const void* v_new, int64_t kv_token_stride,
                          const int64_t* slot_mapping, const void* q, void* out, int32_t max_blocks_per_seq, int32_t batch,
                          int32_t num_q_heads, float sm_scale, int32_t chunk_size, const int32_t* cu_q_lens, void* workspace,
                          int planned_ctas, bool overlap_previous, cudaStream_t stream);
size_t workspace_control_bytes();
int decode_planned_ctas(int num_sms, long long upper_blocks);
int decode_max_batch();
int decode_counter_slots();
int decode_max_chunk_blocks();
void chunk_partial_offsets(int batch, int num_q_heads, int head_dim, int max_chunks, size_t* o, size_t* m, size_t* l);

const DeviceInfo* device_info() {
  static DeviceInfo info[64];
  static bool known[64] = {};
  static std::mutex mu;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(mu);
  if (!known[dev]) {
    int sms = 0, smem = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return nullptr;
    if (cudaDeviceGetAttribute(&smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) return nullptr;
    info[dev].num_sms = sms;
    info[dev].max_smem_optin = smem;
    known[dev] = true;
  }
  return &info[dev];
}

bool configure_kernel_smem(const void* kernel, int bytes) {
  static std::mutex mu;
  static std::vector<std::pair<const void*, int>> done;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return false;
  std::lock_guard<std::mutex> lock(mu);
  for (const auto& d : done)
    if (d.first == kernel && d.second == dev) return true;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
  done.emplace_back(kernel, dev);
  return true;
}

namespace {

bool cache_shape_ok(int head_dim, int block_size, int dtype) {
  return (head_dim == 64 || head_dim == 128) && block_size == kBlockSize &&
         (is_fp8(dtype) || dtype == COOPT_KV_BF16);
}

int check_cache(const coopt_cache* c) {
  if (c == nullptr || c->data == nullptr || c->num_blocks <= 0 || c->num_kv_heads <= 0) return COOPT_ERR_INVALID_ARG;
  if (!cache_shape_ok(c->head_dim, c->block_size, c->dtype)) return COOPT_ERR_UNSUPPORTED;
  if (reinterpret_cast<uintptr_t>(c->data) % 32 != 0) return COOPT_ERR_INVALID_ARG;
  return COOPT_OK;
}

int max_chunks_of(int max_blocks_per_seq, int chunk_size) {
  return static_cast<int>((static_cast<long long>(max_blocks_per_seq) * kBlockSize + chunk_size - 1) / chunk_size);
}

// number of CTAs planned for a decode-style launch; the same on the sizing and the launching side
int planned_ctas(int batch, int num_kv_heads, int max_blocks_per_seq) {
  const DeviceInfo* di = device_info();
  const int sms = di ? di->num_sms : 148;
  return decode_planned_ctas(sms, static_cast<long long>(batch) * num_kv_heads * max_blocks_per_seq);
}

}  // namespace

int check_attention_shapes(const coopt_cache* c, const void* q, void* out, int32_t max_blocks_per_seq, int32_t batch,
                           int32_t num_q_heads);

// Every host-side check of a decode-style call (shared with the entry points of other files).
int check_attention_args(const coopt_cache* c, const void* q, void* out, const int32_t* block_table,
                         int32_t max_blocks_per_seq, const int32_t* context_lens, int32_t batch, int32_t num_q_heads) {
  const int rc = check_attention_shapes(c, q, out, max_blocks_per_seq, batch, num_q_heads);
  if (rc != COOPT_OK) return rc;
  return block_table && context_lens ? COOPT_OK : COOPT_ERR_INVALID_ARG;
}

int check_attention_shapes(const coopt_cache* c, const void* q, void* out, int32_t max_blocks_per_seq, int32_t batch,
                           int32_t num_q_heads) {
  const int rc = check_cache(c);
  if (rc != COOPT_OK) return rc;
  if (!q || !out || batch < 0 || max_blocks_per_seq <= 0 || num_q_heads <= 0) return COOPT_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(out)) % 16 != 0) return COOPT_ERR_INVALID_ARG;   // rows move in 16-byte pieces
  if (num_q_heads % c->num_kv_heads != 0) return COOPT_ERR_UNSUPPORTED;
  const int group = num_q_heads / c->num_kv_heads;
  if (group < 1 || group > 8) return COOPT_ERR_UNSUPPORTED;
  if (batch > decode_max_batch() || static_cast<long long>(batch) * c->num_kv_heads > decode_counter_slots())
    return COOPT_ERR_UNSUPPORTED;
  // the planner indexes (sequence, kv head, block) triples with 31 bits
  if (static_cast<long long>(batch) * c->num_kv_heads * max_blocks_per_seq >= (1ll << 31)) return COOPT_ERR_UNSUPPORTED;
  return COOPT_OK;
}

}  // namespace coopt

using namespace coopt;

extern "C" {

size_t coopt_granule_bytes(int32_t head_dim, int32_t dtype) {
  if (!cache_shape_ok(head_dim, kBlockSize, dtype)) return 0;
  return granule_bytes(head_dim, is_fp8(dtype));
}

size_t coopt_cache_bytes(int32_t num_blocks, int32_t num_kv_heads, int32_t head_dim, int32_t dtype) {
  if (num_blocks <= 0 || num_kv_heads <= 0) return 0;
  return static_cast<size_t>(num_blocks) * num_kv_heads * coopt_granule_bytes(head_dim, dtype);
}

int64_t coopt_cache_offset(const coopt_cache* c, int32_t block, int32_t kv_head, int32_t which, int32_t token,
                           int32_t dim) {
  if (!c || !cache_shape_ok(c->head_dim, c->block_size, c->dtype)) return -1;
  if (block < 0 || block >= c->num_blocks || kv_head < 0 || kv_head >= c->num_kv_heads || which < 0 || which > 1 ||
      token < 0 || token >= kBlockSize || dim < 0 || dim >= c->head_dim)
    return -1;
  const bool fp8 = is_fp8(c->dtype);
  const int64_t gran = (static_cast<int64_t>(block) * c->num_kv_heads + kv_head) * granule_bytes(c->head_dim, fp8);
  const int inner = which == 0 ? k_elem_offset(c->head_dim, fp8, token, dim) : v_elem_offset(c->head_dim, fp8, token, dim);
  return gran + part_offset(c->head_dim, fp8, which) + inner;
}

int64_t coopt_scale_offset(const coopt_cache* c, int32_t block, int32_t kv_head, int32_t which) {
  if (!c || !cache_shape_ok(c->head_dim, c->block_size, c->dtype) || !is_fp8(c->dtype)) return -1;
  if (block < 0 || block >= c->num_blocks || kv_head < 0 || kv_head >= c->num_kv_heads || which < 0 || which > 1) return -1;
  return (static_cast<int64_t>(block) * c->num_kv_heads + kv_head) * granule_bytes(c->head_dim, true) + header_offset(c->head_dim) + 4 * which;
}

int coopt_kv_write(const coopt_cache* cache, const void* k, const void* v, int64_t kv_token_stride,
                   const int64_t* slot_mapping, int32_t num_tokens, void* stream) {
  const int rc = check_cache(cache);
  if (rc != COOPT_OK) return rc;
  if (num_tokens < 0) return COOPT_ERR_INVALID_ARG;
  if (num_tokens == 0) return COOPT_OK;
  if (!k || !v || !slot_mapping) return COOPT_ERR_INVALID_ARG;
  if (kv_token_stride < static_cast<int64_t>(cache->num_kv_heads) * cache->head_dim) return COOPT_ERR_INVALID_ARG;
  return launch_kv_write(cache, k, v, kv_token_stride, slot_mapping, num_tokens, static_cast<cudaStream_t>(stream));
}

size_t coopt_workspace_bytes(int32_t batch, int32_t num_q_heads, int32_t num_kv_heads, int32_t head_dim,
                             int32_t max_blocks_per_seq, int32_t chunk_size, int32_t total_q) {
  (void)total_q;
  if (batch < 0 || num_q_heads <= 0 || num_kv_heads <= 0 || max_blocks_per_seq <= 0 || chunk_size < 0) return 0;
  const int group = (num_q_heads + num_kv_heads - 1) / num_kv_heads;
  const int P = planned_ctas(batch, num_kv_heads, max_blocks_per_seq);
  const int mc = chunk_size > 0 ? max_chunks_of(max_blocks_per_seq, chunk_size) : 0;
  return decode_workspace_bytes(P, group, head_dim, batch, num_q_heads, num_kv_heads, max_blocks_per_seq, chunk_size / kBlockSize, mc);
}

int coopt_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
  if (!workspace) return COOPT_ERR_INVALID_ARG;
  if (workspace_bytes < workspace_control_bytes()) return COOPT_ERR_WORKSPACE;
  return cudaMemsetAsync(workspace, 0, workspace_control_bytes(), static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? COOPT_OK
             : COOPT_ERR_CUDA;
}

int coopt_chunk_partials(int32_t batch, int32_t num_q_heads, int32_t head_dim, int32_t max_blocks_per_seq,
                         int32_t chunk_size, size_t* o_offset, size_t* m_offset, size_t* l_offset, int32_t* max_chunks) {
  if (batch < 0 || num_q_heads <= 0 || head_dim <= 0 || max_blocks_per_seq <= 0 || chunk_size <= 0 ||
      chunk_size % kBlockSize != 0 || !o_offset || !m_offset || !l_offset || !max_chunks)
    return COOPT_ERR_INVALID_ARG;
  *max_chunks = max_chunks_of(max_blocks_per_seq, chunk_size);
  chunk_partial_offsets(batch, num_q_heads, head_dim, *max_chunks, o_offset, m_offset, l_offset);
  return COOPT_OK;
}

int coopt_paged_decode(const coopt_cache* cache, const void* q, void* out, const int32_t* block_table,
                       int32_t max_blocks_per_seq, const int32_t* context_lens, int32_t batch, int32_t num_q_heads,
                       float sm_scale, void* workspace, size_t workspace_bytes, void* stream) {
  const int rc = check_attention_args(cache, q, out, block_table, max_blocks_per_seq, context_lens, batch, num_q_heads);
  if (rc != COOPT_OK) return rc;
  if (batch == 0) return COOPT_OK;
  if (!workspace || workspace_bytes < coopt_workspace_bytes(batch, num_q_heads, cache->num_kv_heads, cache->head_dim,
                                                            max_blocks_per_seq, 0, batch))
    return COOPT_ERR_WORKSPACE;
  const int P = planned_ctas(batch, cache->num_kv_heads, max_blocks_per_seq);
  return launch_paged_decode(cache, q, out, block_table, max_blocks_per_seq, context_lens, batch, num_q_heads, sm_scale,
                             0, nullptr, workspace, P, static_cast<cudaStream_t>(stream));
}

int coopt_decode_step(const coopt_cache* cache, const void* k_new, const void* v_new, int64_t kv_token_stride,
                      const int64_t* slot_mapping, const void* q, void* out, const int32_t* block_table,
                      int32_t max_blocks_per_seq, const int32_t* context_lens, int32_t batch, int32_t num_q_heads,
                      float sm_scale, void* workspace, size_t workspace_bytes, void* stream) {
  // every check of both halves before anything is launched
  int rc = check_attention_args(cache, q, out, block_table, max_blocks_per_seq, context_lens, batch, num_q_heads);
  if (rc != COOPT_OK) return rc;
  if (!k_new || !v_new || !slot_mapping || kv_token_stride < static_cast<int64_t>(cache->num_kv_heads) * cache->head_dim)
    return COOPT_ERR_INVALID_ARG;
  if (batch == 0) return COOPT_OK;
  if (!workspace || workspace_bytes < coopt_workspace_bytes(batch, num_q_heads, cache->num_kv_heads, cache->head_dim,
                                                            max_blocks_per_seq, 0, batch))
    return COOPT_ERR_WORKSPACE;
  rc = launch_kv_write(cache, k_new, v_new, kv_token_stride, slot_mapping, batch, static_cast<cudaStream_t>(stream));
  if (rc != COOPT_OK) return rc;
  const int P = planned_ctas(batch, cache->num_kv_heads, max_blocks_per_seq);
  return launch_paged_decode(cache, q, out, block_table, max_blocks_per_seq, context_lens, batch, num_q_heads, sm_scale,
                             0, nullptr, workspace, P, static_cast<cudaStream_t>(stream));
}

size_t coopt_plan_bytes(int32_t batch, int32_t num_kv_heads, int32_t max_blocks_per_seq, int32_t chunk_size) {
  if (batch <= 0 || num_kv_heads <= 0 || max_blocks_per_seq <= 0 || chunk_size < 0 || chunk_size % kBlockSize != 0) return 0;
  return plan_bytes(planned_ctas(batch, num_kv_heads, max_blocks_per_seq), batch, num_kv_heads, max_blocks_per_seq, chunk_size / kBlockSize);
}

static int check_plan_args(int32_t batch, int32_t num_kv_heads, int32_t max_blocks_per_seq, int32_t chunk_size, const void* plan,
                           size_t plan_bytes_given) {
  if (batch < 0 || num_kv_heads <= 0 || max_blocks_per_seq <= 0) return COOPT_ERR_INVALID_ARG;
  if (chunk_size < 0 || chunk_size % kBlockSize != 0 || chunk_size / kBlockSize > decode_max_chunk_blocks()) return COOPT_ERR_INVALID_ARG;
  if (batch > decode_max_batch() || static_cast<long long>(batch) * num_kv_heads > decode_counter_slots()) return COOPT_ERR_UNSUPPORTED;
  if (static_cast<long long>(batch) * num_kv_heads * max_blocks_per_seq >= (1ll << 31)) return COOPT_ERR_UNSUPPORTED;
  if (batch == 0) return COOPT_OK;
  if (!plan || reinterpret_cast<uintptr_t>(plan) % 16 != 0) return COOPT_ERR_INVALID_ARG;
  if (plan_bytes_given < coopt_plan_bytes(batch, num_kv_heads, max_blocks_per_seq, chunk_size)) return COOPT_ERR_WORKSPACE;
  return COOPT_OK;
}

int coopt_decode_plan(const int32_t* block_table, int32_t max_blocks_per_seq, const int32_t* context_lens, int32_t batch,
                      int32_t num_kv_heads, int32_t num_blocks, int32_t chunk_size, void* plan, size_t plan_bytes_given,
                      void* stream) {
  const int rc = check_plan_args(batch, num_kv_heads, max_blocks_per_seq, chunk_size, plan, plan_bytes_given);
  if (rc != COOPT_OK) return rc;
  if (!block_table || !context_lens || num_blocks <= 0) return COOPT_ERR_INVALID_ARG;
  if (batch == 0) return COOPT_OK;
  return launch_decode_plan(block_table, max_blocks_per_seq, context_lens, batch, num_kv_heads, num_blocks, chunk_size,
                            planned_ctas(batch, num_kv_heads, max_blocks_per_seq), plan, static_cast<cudaStream_t>(stream));
}

int coopt_decode_step_planned(const coopt_cache* cache, const void* plan, size_t plan_bytes_given, const void* k_new,
                              const void* v_new, int64_t kv_token_stride, const int64_t* slot_mapping, const void* q, void* out,
                              int32_t max_blocks_per_seq, int32_t batch, int32_t num_q_heads, int32_t chunk_size, float sm_scale,
                              void* workspace, size_t workspace_bytes, uint32_t flags, void* stream) {
  int rc = check_attention_shapes(cache, q, out, max_blocks_per_seq, batch, num_q_heads);
  if (rc != COOPT_OK) return rc;
  if (!is_fp8(cache->dtype)) return COOPT_ERR_UNSUPPORTED;                     // the bf16 ablation kernel plans for itself
  rc = check_plan_args(batch, cache->num_kv_heads, max_blocks_per_seq, chunk_size, plan, plan_bytes_given);
  if (rc != COOPT_OK) return rc;
  const bool append = k_new || v_new || slot_mapping;
  if (append && (!k_new || !v_new || !slot_mapping || kv_token_stride < static_cast<int64_t>(cache->num_kv_heads) * cache->head_dim))
    return COOPT_ERR_INVALID_ARG;
  if ((flags & ~static_cast<uint32_t>(COOPT_FLAG_OVERLAP_PREVIOUS)) != 0) return COOPT_ERR_INVALID_ARG;
  if (batch == 0) return COOPT_OK;
  if (!workspace || workspace_bytes < coopt_workspace_bytes(batch, num_q_heads, cache->num_kv_heads, cache->head_dim,
                                                            max_blocks_per_seq, chunk_size, batch))
    return COOPT_ERR_WORKSPACE;
  return launch_decode_planned(cache, plan, k_new, v_new, kv_token_stride, slot_mapping, q, out, max_blocks_per_seq, batch,
                               num_q_heads, sm_scale, chunk_size, nullptr, workspace,
                               planned_ctas(batch, cache->num_kv_heads, max_blocks_per_seq),
                               (flags & COOPT_FLAG_OVERLAP_PREVIOUS) != 0, static_cast<cudaStream_t>(stream));
}

int coopt_decode_layers(const coopt_layer_io* layers, int32_t num_layers, int64_t kv_token_stride, const int32_t* block_table,
                        int32_t max_blocks_per_seq, const int32_t* context_lens, int32_t batch, int32_t num_q_heads,
                        float sm_scale, void* plan, size_t plan_bytes_given, void* workspace, size_t workspace_bytes,
                        uint32_t flags, void* stream) {
  if (!layers || num_layers <= 0) return COOPT_ERR_INVALID_ARG;
  // every check of every layer before anything is launched
  const coopt_cache* c0 = layers[0].cache;
  for (int32_t l = 0; l < num_layers; ++l) {
    const coopt_layer_io& io = layers[l];
    const int rc = check_attention_shapes(io.cache, io.q, io.out, max_blocks_per_seq, batch, num_q_heads);
    if (rc != COOPT_OK) return rc;
    if (!is_fp8(io.cache->dtype) || io.cache->dtype != c0->dtype) return COOPT_ERR_UNSUPPORTED;
    if (io.cache->num_kv_heads != c0->num_kv_heads || io.cache->head_dim != c0->head_dim || io.cache->num_blocks != c0->num_blocks)
      return COOPT_ERR_INVALID_ARG;                                             // one plan serves every layer
    const bool append = io.k_new || io.v_new || io.slot_mapping;
    if (append && (!io.k_new || !io.v_new || !io.slot_mapping || kv_token_stride < static_cast<int64_t>(c0->num_kv_heads) * c0->head_dim))
      return COOPT_ERR_INVALID_ARG;
  }
  int rc = check_plan_args(batch, c0->num_kv_heads, max_blocks_per_seq, 0, plan, plan_bytes_given);
  if (rc != COOPT_OK) return rc;
  if (!block_table || !context_lens) return COOPT_ERR_INVALID_ARG;
  if ((flags & ~static_cast<uint32_t>(COOPT_FLAG_OVERLAP_PREVIOUS)) != 0) return COOPT_ERR_INVALID_ARG;
  if (batch == 0) return COOPT_OK;
  if (!workspace || workspace_bytes < coopt_workspace_bytes(batch, num_q_heads, c0->num_kv_heads, c0->head_dim, max_blocks_per_seq, 0, batch))
    return COOPT_ERR_WORKSPACE;
  const int P = planned_ctas(batch, c0->num_kv_heads, max_blocks_per_seq);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  rc = launch_decode_plan(block_table, max_blocks_per_seq, context_lens, batch, c0->num_kv_heads, c0->num_blocks, 0, P, plan, st);
  for (int32_t l = 0; l < num_layers && rc == COOPT_OK; ++l) {
    const coopt_layer_io& io = layers[l];
    // layer l > 0 may start while layer l - 1 drains: its copy warp reads only the plan and its own cache
    rc = launch_decode_planned(io.cache, plan, io.k_new, io.v_new, kv_token_stride, io.slot_mapping, io.q, io.out, max_blocks_per_seq,
                               batch, num_q_heads, sm_scale, 0, nullptr, workspace, P,
                               l > 0 && (flags & COOPT_FLAG_OVERLAP_PREVIOUS) != 0, st);
  }
  return rc;
}

int coopt_paged_chunked(const coopt_cache* cache, const void* q, void* out, const int32_t* cu_q_lens,
                        const int32_t* block_table, int32_t max_blocks_per_seq, const int32_t* context_lens,
                        int32_t batch, int32_t num_q_heads, int32_t total_q, int32_t chunk_size, int32_t causal,
                        float sm_scale, void* workspace, size_t workspace_bytes, void* stream) {
  const int rc = check_attention_args(cache, q, out, block_table, max_blocks_per_seq, context_lens, batch, num_q_heads);
  if (rc != COOPT_OK) return rc;
  if (!cu_q_lens || total_q < batch) return COOPT_ERR_INVALID_ARG;
  if (chunk_size <= 0 || chunk_size % kBlockSize != 0 || chunk_size / kBlockSize > decode_max_chunk_blocks())
    return COOPT_ERR_INVALID_ARG;
  if (batch == 0) return COOPT_OK;
  if (!workspace || workspace_bytes < coopt_workspace_bytes(batch, num_q_heads, cache->num_kv_heads, cache->head_dim,
                                                            max_blocks_per_seq, chunk_size, total_q))
    return COOPT_ERR_WORKSPACE;
  if (total_q == batch) {
    // one query token per sequence: the Opt-Pa chunk-and-merge decode
    const int P = planned_ctas(batch, cache->num_kv_heads, max_blocks_per_seq);
    return launch_paged_decode(cache, q, out, block_table, max_blocks_per_seq, context_lens, batch, num_q_heads,
                               sm_scale, chunk_size, cu_q_lens, workspace, P, static_cast<cudaStream_t>(stream));
  }
  return launch_paged_prefill(cache, q, out, cu_q_lens, block_table, max_blocks_per_seq, context_lens, batch,
                              num_q_heads, total_q, causal, sm_scale, workspace, static_cast<cudaStream_t>(stream));
}

namespace {
// The device's address of a host pointer if the memory is page-locked and mapped (cudaHostAlloc, cudaHostRegister),
// null for pageable memory (and for anything that is not host memory).
const uint8_t* mapped_host_pointer(const void* host) {
  cudaPointerAttributes attr;
  if (cudaPointerGetAttributes(&attr, host) != cudaSuccess) {
    (void)cudaGetLastError();
    return nullptr;
  }
  if (attr.type != cudaMemoryTypeHost || attr.devicePointer == nullptr) return nullptr;
  return static_cast<const uint8_t*>(attr.devicePointer);
}

coopt_step_layout step_layout(int batch, int hq, int hkv, int d, int max_blocks) {
  auto up = [](size_t x) { return (x + 255) / 256 * 256; };
  coopt_step_layout s;
  size_t at = 0;
  s.q = at;            at += up(static_cast<size_t>(batch) * hq * d * 2);
  s.k_new = at;        at += up(static_cast<size_t>(batch) * hkv * d * 2);
  s.v_new = at;        at += up(static_cast<size_t>(batch) * hkv * d * 2);
  s.slot_mapping = at; at += up(static_cast<size_t>(batch) * 8);
  s.block_table = at;  at += up(static_cast<size_t>(batch) * max_blocks * 4);
  s.context_lens = at; at += up(static_cast<size_t>(batch) * 4);
  s.in_bytes = at;
  s.out = at;          at += up(static_cast<size_t>(batch) * hq * d * 2);
  s.out_bytes = static_cast<size_t>(batch) * hq * d * 2;
  s.total_bytes = at;
  return s;
}
}  // namespace

int coopt_step_staging_layout(int32_t batch, int32_t num_q_heads, int32_t num_kv_heads, int32_t head_dim,
                              int32_t max_blocks_per_seq, coopt_step_layout* layout) {
  if (batch < 0 || num_q_heads <= 0 || num_kv_heads <= 0 || head_dim <= 0 || max_blocks_per_seq <= 0 || !layout) return COOPT_ERR_INVALID_ARG;
  *layout = step_layout(batch, num_q_heads, num_kv_heads, head_dim, max_blocks_per_seq);
  return COOPT_OK;
}

int coopt_decode_step_host(const coopt_cache* cache, const void* step_inputs_host, void* out_host, int32_t max_blocks_per_seq,
                           int32_t batch, int32_t num_q_heads, float sm_scale, void* staging, size_t staging_bytes, void* plan,
                           size_t plan_bytes_given, void* workspace, size_t workspace_bytes, void* stream) {
  int rc = check_cache(cache);
  if (rc != COOPT_OK) return rc;
  if (!step_inputs_host || !out_host || batch < 0 || num_q_heads <= 0 || max_blocks_per_seq <= 0) return COOPT_ERR_INVALID_ARG;
  if (batch == 0) return COOPT_OK;
  const int hkv = cache->num_kv_heads, d = cache->head_dim;
  const coopt_step_layout s = step_layout(batch, num_q_heads, hkv, d, max_blocks_per_seq);
  if (!staging || staging_bytes < s.total_bytes) return COOPT_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(staging) % 256 != 0) return COOPT_ERR_INVALID_ARG;
  uint8_t* dev = static_cast<uint8_t*>(staging);
  // every check of the device part before the first copy is enqueued
  rc = check_attention_args(cache, dev + s.q, dev + s.out, reinterpret_cast<const int32_t*>(dev + s.block_table), max_blocks_per_seq,
                            reinterpret_cast<const int32_t*>(dev + s.context_lens), batch, num_q_heads);
  if (rc != COOPT_OK) return rc;
  if (!is_fp8(cache->dtype)) return COOPT_ERR_UNSUPPORTED;
  rc = check_plan_args(batch, hkv, max_blocks_per_seq, 0, plan, plan_bytes_given);
  if (rc != COOPT_OK) return rc;
  if (!workspace || workspace_bytes < coopt_workspace_bytes(batch, num_q_heads, hkv, d, max_blocks_per_seq, 0, batch)) return COOPT_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int P = planned_ctas(batch, hkv, max_blocks_per_seq);
  // Host buffers that are page-locked and mapped into the device's address space are used where they are: the
  // kernel fetches the queries and the new tokens from them and stores the result into them, and only the
  // index arrays (slots, block table, context lengths: what the planner walks) are copied to the device.
  const uint8_t* in_dev = mapped_host_pointer(step_inputs_host);
  uint8_t* out_dev = const_cast<uint8_t*>(mapped_host_pointer(out_host));
  if (in_dev != nullptr && out_dev != nullptr && reinterpret_cast<uintptr_t>(in_dev) % 16 == 0 && reinterpret_cast<uintptr_t>(out_dev) % 16 == 0) {
    if (cudaMemcpyAsync(dev + s.slot_mapping, static_cast<const uint8_t*>(step_inputs_host) + s.slot_mapping, s.in_bytes - s.slot_mapping,
                        cudaMemcpyHostToDevice, st) != cudaSuccess)
      return COOPT_ERR_CUDA;
    rc = launch_decode_plan(reinterpret_cast<const int32_t*>(dev + s.block_table), max_blocks_per_seq,
                            reinterpret_cast<const int32_t*>(dev + s.context_lens), batch, hkv, cache->num_blocks, 0, P, plan, st);
    if (rc != COOPT_OK) return rc;
    return launch_decode_planned(cache, plan, in_dev + s.k_new, in_dev + s.v_new, static_cast<int64_t>(hkv) * d,
                                 reinterpret_cast<const int64_t*>(dev + s.slot_mapping), in_dev + s.q, out_dev, max_blocks_per_seq,
                                 batch, num_q_heads, sm_scale, 0, nullptr, workspace, P, false, st);
  }
  // pageable host memory: one copy in, the plan and the fused step, one copy out
  if (cudaMemcpyAsync(dev, step_inputs_host, s.in_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return COOPT_ERR_CUDA;
  rc = launch_decode_plan(reinterpret_cast<const int32_t*>(dev + s.block_table), max_blocks_per_seq,
                          reinterpret_cast<const int32_t*>(dev + s.context_lens), batch, hkv, cache->num_blocks, 0, P, plan, st);
  if (rc != COOPT_OK) return rc;
  rc = launch_decode_planned(cache, plan, dev + s.k_new, dev + s.v_new, static_cast<int64_t>(hkv) * d,
                             reinterpret_cast<const int64_t*>(dev + s.slot_mapping), dev + s.q, dev + s.out, max_blocks_per_seq, batch,
                             num_q_heads, sm_scale, 0, nullptr, workspace, P, false, st);
  if (rc != COOPT_OK) return rc;
  return cudaMemcpyAsync(out_host, dev + s.out, s.out_bytes, cudaMemcpyDeviceToHost, st) == cudaSuccess ? COOPT_OK : COOPT_ERR_CUDA;
}

const char* coopt_status_string(int status) {
  switch (status) {
    case COOPT_OK: return "ok";
    case COOPT_ERR_INVALID_ARG: return "invalid argument";
    case COOPT_ERR_UNSUPPORTED: return "unsupported shape";
    case COOPT_ERR_WORKSPACE: return "workspace missing or too small";
    case COOPT_ERR_CUDA: return "CUDA runtime error";
    case COOPT_ERR_TIMEOUT: return "device-side wait timed out";
    default: return "unknown status";
  }
}

int coopt_version(void) { return 200; }

}  // extern "C"
