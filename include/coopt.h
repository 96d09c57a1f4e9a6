/*
 * coopt.h — C ABI of the paged FP8 grouped-query attention library (libcoopt.so).
 *
 * One attention layer's hot path of LLM-CoOpt: the Opt-KV cache write (Algorithm 1,
 * phase 1), the Opt-KV / Opt-GQA read (Algorithm 1 phase 2, Algorithm 2, Eq. 6-8) and the
 * Opt-Pa valid-block / chunk-and-merge path (Algorithm 3, Eq. 9-10).  sm_100a only; there
 * is no CPU fallback.
 *
 * General rules for every call
 *   - Pointers marked DEVICE must point to memory of the current CUDA device; the caller
 *     owns all of it.  The library allocates no device memory and never synchronises: work
 *     is enqueued on `stream` (a cudaStream_t passed as void*; NULL = the default stream).
 *   - The return value is a coopt_status: 0 on success, negative after host-side argument
 *     checks or a failed launch.  Nothing is thrown, nothing aborts.
 *   - Problems seen on the device (a bounded wait that ran out) are reported in the first
 *     int32 of the workspace (0 = none, otherwise a coopt_status); read it after the
 *     stream has been synchronised.
 *
 * Cache layout (DEVICE memory, `coopt_cache.data`)
 *   The cache is an array of granules, one per (physical block, kv head):
 *       granule(blk, h) starts at byte (blk * num_kv_heads + h) * coopt_granule_bytes().
 *   block_size is 16 tokens.  FP8 E4M3 cache (COOPT_KV_FP8_E4M3), D = head_dim:
 *       bytes 0..16*D-1        K codes: token t, dim d at (t/8)*8D + (d/16)*128 + (t%8)*16 + d%16
 *       bytes 16*D..32*D-1     V codes, transposed: token t, dim d at (d/8)*128 + (d%8)*16 + t
 *       bytes 32*D..32*D+3     fp32 K scale of the granule     bytes 32*D+4..32*D+7  fp32 V scale
 *       bytes 32*D+8..32*D+31  zero
 *       bytes 32*D+32..32*D+127 padding (never read, never written: a granule is 32*D + 128 bytes, so that
 *                              granules start on 128-byte lines)
 *   A dequantised element is decode_e4m3(code) * scale (Eq. 6).  A scale of 0 marks a
 *   granule that holds only zeros.  Both parts are laid out as the tensor cores read matrix
 *   operands from shared memory (8 rows x 16 bytes form one contiguous 128-byte unit), so a part
 *   needs one copy and no rearrangement on its way from HBM to the matrix instruction.
 *   bf16 cache (COOPT_KV_BF16, the un-quantised ablation): no header; 16*D bf16 K values then
 *   16*D bf16 V values, permuted into the register order of the warp-level matrix instruction.
 *   coopt_cache_offset() returns the byte offset of any element, which is all a caller needs to
 *   inspect or build a cache by hand.  Slots of a block past the context should hold finite codes.
 *   A cache that has never been written must be zero-filled once by the caller.
 */
#ifndef COOPT_H_
#define COOPT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  COOPT_OK = 0,
  COOPT_ERR_INVALID_ARG = -1, /* null pointer, negative size, inconsistent shapes       */
  COOPT_ERR_UNSUPPORTED = -2, /* shape outside the compiled set (see each call)          */
  COOPT_ERR_WORKSPACE = -3,   /* workspace missing or smaller than coopt_workspace_bytes */
  COOPT_ERR_CUDA = -4,        /* a CUDA runtime call or the launch failed                */
  COOPT_ERR_TIMEOUT = -5      /* device side: a bounded wait ran out (workspace word 0)  */
} coopt_status;

/* COOPT_KV_FP8_E5M2 is an ablation of the FP8 format, which Section 3.1 leaves open: the same granule layout and the
 * same scale rule with codes in the OCP E5M2 format (5 exponent bits, 2 mantissa bits, saturating at +-57344:
 * scale = amax / 57344).  Supported by every call except chunked prefill at head_dim 64. */
typedef enum { COOPT_KV_FP8_E4M3 = 0, COOPT_KV_BF16 = 1, COOPT_KV_FP8_E5M2 = 2 } coopt_kv_dtype;

typedef struct coopt_cache {
  void* data;           /* DEVICE, coopt_cache_bytes() bytes, 32-byte aligned, layout above */
  int32_t num_blocks;   /* physical blocks                                                 */
  int32_t num_kv_heads; /* H_k of Eq. 7                                                    */
  int32_t head_dim;     /* 64 or 128                                                       */
  int32_t block_size;   /* must be 16                                                      */
  int32_t dtype;        /* coopt_kv_dtype                                                  */
} coopt_cache;

/* Bytes of one (block, kv head) granule / of a whole cache; 0 for unsupported shapes. */
size_t coopt_granule_bytes(int32_t head_dim, int32_t dtype);
size_t coopt_cache_bytes(int32_t num_blocks, int32_t num_kv_heads, int32_t head_dim, int32_t dtype);

/* Byte offset, from `data`, of element (block, kv_head, which, token, dim); which = 0 for K,
 * 1 for V.  For the FP8 cache the granule's K (V) scale is at coopt_scale_offset(..., which).
 * Pure host arithmetic (no CUDA call); returns -1 for arguments out of range. */
int64_t coopt_cache_offset(const coopt_cache* cache, int32_t block, int32_t kv_head, int32_t which,
                           int32_t token, int32_t dim);
int64_t coopt_scale_offset(const coopt_cache* cache, int32_t block, int32_t kv_head, int32_t which);

/*
 * coopt_kv_write — Opt-KV write (Algorithm 1 phase 1; Eq. 5; Section 3.1 "compressing
 * valid blocks into FP8").
 *   k, v          DEVICE bf16 [num_tokens][num_kv_heads][head_dim]; consecutive tokens are
 *                 kv_token_stride elements apart (>= num_kv_heads * head_dim)
 *   slot_mapping  DEVICE int64 [num_tokens]; slot = block * 16 + offset.  A negative slot
 *                 skips the token (Eq. 5; the caller expresses SkipSet membership this way).
 * FP8 semantics, per group of the call's tokens that land in one block, per kv head and
 * for K and V separately: amax = largest |value| of the group; a group that writes offset 0
 * opens the block anew (old scale ignored, all other slots cleared to code 0); otherwise
 * s_old is the granule's scale.  s_new = max(s_old, amax / 448).  If s_new > s_old > 0 the
 * codes already in the granule are re-expressed: enc((dec(code) * s_old) / s_new).  New
 * values are stored as enc(x / s_new).  All of this in IEEE fp32; enc is round-to-nearest-
 * even with saturation to +-448.  bf16 cache: values are stored unchanged.
 * Preconditions (not checked): inputs finite; the non-skipped tokens of one call that land
 * in the same block are consecutive in the call (skipped tokens may sit between them) and
 * have distinct offsets; no other work touches those blocks concurrently.  Tokens whose
 * block index is >= num_blocks are ignored.
 * Errors: INVALID_ARG (null pointers, num_tokens < 0, stride too small), UNSUPPORTED
 * (head_dim not 64/128, block_size != 16, unknown dtype), CUDA.  num_tokens == 0 is a no-op.
 */
int coopt_kv_write(const coopt_cache* cache, const void* k, const void* v, int64_t kv_token_stride,
                   const int64_t* slot_mapping, int32_t num_tokens, void* stream);

/*
 * coopt_paged_decode — one new query token per sequence attends over its paged cache
 * (Eq. 1; Eq. 6 dequantisation on load; Eq. 7-8 grouped-query sharing: query head i reads
 * kv head floor(i / (num_q_heads / num_kv_heads)); Eq. 9: only blocks 0..ceil(len/16)-1 of a
 * sequence are read and the last one is masked past len; Eq. 10 max-subtracted softmax).
 *   q, out        DEVICE bf16 [batch][num_q_heads][head_dim], contiguous, 16-byte aligned
 *   block_table   DEVICE int32 [batch][max_blocks_per_seq]; entry j of row b is the physical
 *                 block of tokens 16j..16j+15 of sequence b; entries past the context are
 *                 never read
 *   context_lens  DEVICE int32 [batch]; 0 gives an all-zero output row
 *   sm_scale      logit scale, normally 1/sqrt(head_dim)
 *   workspace     DEVICE, >= coopt_workspace_bytes(...) with chunk_size = 0, prepared once by
 *                 coopt_workspace_init(); reusable by later calls on the same stream
 * The context of every (sequence, kv head) is cut into byte-balanced pieces across the SMs;
 * pieces are merged by a log-sum-exp reduction inside the same launch.  The cut is planned by a
 * small launch of its own in front of the attention kernel (into the workspace); callers that run
 * many layers per step plan once with coopt_decode_plan instead.
 * Errors: INVALID_ARG, UNSUPPORTED (group size num_q_heads/num_kv_heads not in 1..8 or not
 * integral, batch > 512, head_dim/block_size/dtype as above), WORKSPACE, CUDA.
 */
int coopt_paged_decode(const coopt_cache* cache, const void* q, void* out, const int32_t* block_table,
                       int32_t max_blocks_per_seq, const int32_t* context_lens, int32_t batch,
                       int32_t num_q_heads, float sm_scale, void* workspace, size_t workspace_bytes,
                       void* stream);

/*
 * coopt_paged_decode_static -- coopt_paged_decode without a caller-provided workspace.  (The
 * paper has no counterpart of this call; the result is the one coopt_paged_decode gives.)
 * It exists for callers that cannot allocate device memory where they call from: a plug-in
 * whose enqueue hook must not allocate, a server that handed all device memory to its own
 * pool at start-up so that a later cudaMalloc would fail or stall the device, a C program
 * without a device allocator.  The split-KV partials and control words go to a fixed array of
 * COOPT_STATIC_SCRATCH_BYTES inside the library; every device that loads the library holds
 * that much memory until the process exits.  The call itself allocates nothing.
 *   - Arguments as coopt_paged_decode, minus the workspace.
 *   - Problems whose coopt_workspace_bytes(..., chunk_size = 0) exceeds
 *     COOPT_STATIC_SCRATCH_BYTES are refused with COOPT_ERR_WORKSPACE before anything is
 *     enqueued (the LLaMA-13B decode shape needs about 0.8 MB).
 *   - The first call on a device looks up the array's device address; make that first call
 *     outside any stream capture.
 *   - All calls on a device share the array.  Each call clears the control words on `stream`
 *     before its launch, so calls ordered on one stream are safe back to back; calls that can
 *     overlap on the GPU (different streams, different host threads) race on the array and
 *     must be serialised by the caller.
 *   - The device-side status word lives in the array and is not visible to the caller; use
 *     coopt_paged_decode where it must be read.
 */
#define COOPT_STATIC_SCRATCH_BYTES (4 * 1024 * 1024)
int coopt_paged_decode_static(const coopt_cache* cache, const void* q, void* out, const int32_t* block_table,
                              int32_t max_blocks_per_seq, const int32_t* context_lens, int32_t batch,
                              int32_t num_q_heads, float sm_scale, void* stream);

/*
 * coopt_paged_chunked — Opt-Pa long-sequence path (abstract and conclusion: the context is
 * segmented into chunks that are processed independently and merged) and chunked prefill.
 *   cu_q_lens     DEVICE int32 [batch + 1], prefix sums of the number of query tokens per
 *                 sequence; q/out are bf16 [cu_q_lens[batch]][num_q_heads][head_dim]
 *   context_lens  include the new tokens; the n query tokens of a sequence are its last n
 *                 positions and, when causal != 0, query i sees positions 0..len-n+i
 *   chunk_size    tokens per chunk, a multiple of 16, at most 32768
 *   total_q       cu_q_lens[batch] as known by the host (sizes the launch)
 * Precondition when total_q == batch: every sequence has exactly one query token, i.e. cu_q_lens is
 * 0, 1, .., batch (any other split of the same total is reported as COOPT_ERR_INVALID_ARG in the
 * workspace status word and the output is then meaningless).
 * When every sequence has exactly one query token (total_q == batch) each chunk c of
 * (sequence b, query head h) produces m_c (max logit, natural-log units after sm_scale),
 * l_c (sum of exp(logit - m_c)) and o_c (softmax-weighted V inside the chunk, fp32), stored
 * in the workspace where coopt_chunk_partials() points, and the chunks are merged with
 * weights l_c * exp(m_c - max_c m_c).  With longer query runs (chunked prefill) the tiles
 * run on tensor cores and no partials are exported.
 * Errors: as coopt_paged_decode, plus INVALID_ARG for a bad chunk_size.
 */
int coopt_paged_chunked(const coopt_cache* cache, const void* q, void* out, const int32_t* cu_q_lens,
                        const int32_t* block_table, int32_t max_blocks_per_seq, const int32_t* context_lens,
                        int32_t batch, int32_t num_q_heads, int32_t total_q, int32_t chunk_size, int32_t causal,
                        float sm_scale, void* workspace, size_t workspace_bytes, void* stream);

/*
 * coopt_decode_step — one serving step with DEVICE inputs (Algorithm 1: phase 1, the new token of
 * every sequence is written to the cache; phase 2 and Algorithms 2-3, attention over the updated
 * cache): coopt_kv_write(k_new, v_new, slot_mapping, num_tokens = batch) followed by
 * coopt_paged_decode, with the same arguments, results and errors as those two calls made one after
 * the other, in one call.
 *   k_new, v_new   DEVICE bf16 [batch][num_kv_heads][head_dim], kv_token_stride elements apart
 *   slot_mapping   DEVICE int64 [batch]
 *   context_lens   DEVICE int32 [batch], counting the new token
 * All arguments are checked before anything is launched.
 */
int coopt_decode_step(const coopt_cache* cache, const void* k_new, const void* v_new, int64_t kv_token_stride,
                      const int64_t* slot_mapping, const void* q, void* out, const int32_t* block_table,
                      int32_t max_blocks_per_seq, const int32_t* context_lens, int32_t batch, int32_t num_q_heads,
                      float sm_scale, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Planned decode: the work decomposition of a decode step depends only on the context lengths and the
 * block table, which every layer of a model shares within one step (the decode loop of Section 2 visits
 * the same sequences once per layer; Eq. 9's valid blocks are the same in each).  coopt_decode_plan
 * computes it once -- every CTA's share of the (sequence, kv head, block) list with the physical block
 * ids looked up and range-checked -- and coopt_decode_step_planned / coopt_decode_layers read it in
 * every launch instead of working it out again.
 *
 * coopt_plan_bytes      bytes of a plan buffer for these shapes (host arithmetic; 0 for bad arguments).
 * coopt_decode_plan     fills `plan` (DEVICE, 16-byte aligned, >= coopt_plan_bytes) on `stream`.
 *   block_table, context_lens   DEVICE, as for coopt_paged_decode; context_lens count the token a following
 *                               step appends
 *   num_blocks                  of the caches the plan will be used with (block ids are checked against it;
 *                               a bad id is replaced by 0 and reported by the launches that use the plan)
 *   chunk_size                  0 for decode; the chunk size of an Opt-Pa chunked call otherwise
 * Errors: INVALID_ARG, UNSUPPORTED (batch > 512 and the other limits of coopt_paged_decode), WORKSPACE
 * (plan buffer too small), CUDA.
 */
size_t coopt_plan_bytes(int32_t batch, int32_t num_kv_heads, int32_t max_blocks_per_seq, int32_t chunk_size);
int coopt_decode_plan(const int32_t* block_table, int32_t max_blocks_per_seq, const int32_t* context_lens, int32_t batch,
                      int32_t num_kv_heads, int32_t num_blocks, int32_t chunk_size, void* plan, size_t plan_bytes,
                      void* stream);

/*
 * coopt_decode_step_planned -- Algorithm 1 in ONE launch: phase 1 (the new token of every sequence is
 * compressed to FP8 and stored, Eq. 5 skip rule, dynamic per-block scales exactly as coopt_kv_write) and
 * phase 2 with Algorithms 2-3 (attention over the updated cache, exactly as coopt_paged_decode).  The CTA
 * whose share of the plan holds the last block of a (sequence, kv head) writes that sequence's new token
 * into it before its copy engine requests the block; no other CTA reads that block.
 *   plan                       DEVICE, made by coopt_decode_plan for the same batch, num_kv_heads,
 *                              max_blocks_per_seq, chunk_size and num_blocks (a mismatch is reported as
 *                              COOPT_ERR_INVALID_ARG in the workspace status word and the launch does nothing)
 *   k_new, v_new, slot_mapping DEVICE, as for coopt_decode_step; all three NULL = nothing is appended.
 *                              Precondition: the new token of sequence b is its last position, i.e.
 *                              slot_mapping[b] / 16 is the block-table entry of position context_lens[b] - 1
 *                              and slot_mapping[b] % 16 == (context_lens[b] - 1) % 16 (else INVALID_ARG in the
 *                              status word); sequences with slot_mapping[b] < 0 are not written (Eq. 5)
 *   chunk_size                 0, or the plan's chunk size: per-chunk partials as coopt_paged_chunked
 *   flags                      COOPT_FLAG_OVERLAP_PREVIOUS: the launch may start while the kernel before it
 *                              in the stream still runs.  The caller guarantees that this kernel writes neither
 *                              the plan nor this cache; everything else the step reads or writes (q, k_new,
 *                              v_new, slot_mapping, out, workspace) is touched only after that kernel has
 *                              finished.
 * Results: cache bytes and output identical to coopt_kv_write followed by coopt_paged_decode.
 * Errors: as coopt_paged_decode, plus UNSUPPORTED for a bf16 cache.
 */
#define COOPT_FLAG_OVERLAP_PREVIOUS 1u
int coopt_decode_step_planned(const coopt_cache* cache, const void* plan, size_t plan_bytes, const void* k_new,
                              const void* v_new, int64_t kv_token_stride, const int64_t* slot_mapping, const void* q, void* out,
                              int32_t max_blocks_per_seq, int32_t batch, int32_t num_q_heads, int32_t chunk_size, float sm_scale,
                              void* workspace, size_t workspace_bytes, uint32_t flags, void* stream);

/*
 * coopt_decode_layers -- the decode loop of Section 2 over the layers of a model for one step: one plan,
 * then one coopt_decode_step_planned launch per layer, enqueued back to back on `stream`.
 *   layers        HOST array of num_layers entries; every pointer inside is DEVICE memory: the layer's cache
 *                 (all of one shape), its new token's k/v and slots (all NULL = no append), its q and out
 *   block_table, context_lens, plan, workspace   shared by all layers
 *   flags         COOPT_FLAG_OVERLAP_PREVIOUS lets layer l + 1 start while layer l drains (its copy engine
 *                 reads only the plan and its own cache until layer l has finished)
 * Errors: as the calls it makes; every argument of every layer is checked before anything is launched.
 */
typedef struct coopt_layer_io {
  const coopt_cache* cache;
  const void* k_new;            /* DEVICE bf16 [batch][num_kv_heads][head_dim] or NULL */
  const void* v_new;
  const int64_t* slot_mapping;  /* DEVICE int64 [batch] or NULL */
  const void* q;                /* DEVICE bf16 [batch][num_q_heads][head_dim] */
  void* out;
} coopt_layer_io;
int coopt_decode_layers(const coopt_layer_io* layers, int32_t num_layers, int64_t kv_token_stride, const int32_t* block_table,
                        int32_t max_blocks_per_seq, const int32_t* context_lens, int32_t batch, int32_t num_q_heads,
                        float sm_scale, void* plan, size_t plan_bytes, void* workspace, size_t workspace_bytes,
                        uint32_t flags, void* stream);

/*
 * coopt_decode_step_host -- one serving step for callers whose step inputs live in HOST memory (Section 2's
 * token-insertion phase followed by the attention phase).  If both host buffers are page-locked and mapped
 * (cudaHostAlloc, cudaHostRegister; 16-byte aligned), the kernel reads the queries and the new tokens from
 * them and stores the bf16 result into them directly, and only the index arrays (slots, block table, context
 * lengths) are copied to the device for coopt_decode_plan.  Otherwise ONE copy brings the step's inputs to the
 * device, the plan and the step run on them, and ONE copy takes the result back.  Results are identical either
 * way.  Everything is enqueued on `stream`; the host buffers must stay valid until the stream has been
 * synchronised, and out_host holds the result only then.
 *   step_inputs_host   HOST, coopt_step_layout.in_bytes bytes: the step's inputs packed at the offsets that
 *                      coopt_step_staging_layout() gives -- q bf16 [batch][num_q_heads][head_dim]; k_new,
 *                      v_new bf16 [batch][num_kv_heads][head_dim]; slot_mapping int64 [batch]; block_table
 *                      int32 [batch][max_blocks_per_seq]; context_lens int32 [batch], counting the new token
 *   out_host           HOST bf16 [batch][num_q_heads][head_dim]
 *   staging            DEVICE, >= coopt_step_layout.total_bytes, 256-byte aligned
 *   plan, workspace    DEVICE, sized by coopt_plan_bytes / coopt_workspace_bytes (chunk_size 0)
 * The new token of every sequence must be its last position (see coopt_decode_step_planned).
 * Errors: as coopt_decode_plan and coopt_decode_step_planned; WORKSPACE if staging is too small.
 */
typedef struct coopt_step_layout {
  size_t q, k_new, v_new, slot_mapping, block_table, context_lens;   /* byte offsets of the inputs */
  size_t in_bytes;       /* bytes of the packed inputs = what is copied to the device */
  size_t out;            /* byte offset of the result inside the device staging area */
  size_t out_bytes;      /* bytes copied back */
  size_t total_bytes;    /* bytes of the device staging area */
} coopt_step_layout;
int coopt_step_staging_layout(int32_t batch, int32_t num_q_heads, int32_t num_kv_heads, int32_t head_dim,
                              int32_t max_blocks_per_seq, coopt_step_layout* layout);
int coopt_decode_step_host(const coopt_cache* cache, const void* step_inputs_host, void* out_host, int32_t max_blocks_per_seq,
                           int32_t batch, int32_t num_q_heads, float sm_scale, void* staging, size_t staging_bytes, void* plan,
                           size_t plan_bytes, void* workspace, size_t workspace_bytes, void* stream);

/* Workspace size for a call with these arguments (chunk_size = 0 for coopt_paged_decode).
 * Host arithmetic only (it asks the current device for its SM count once). */
size_t coopt_workspace_bytes(int32_t batch, int32_t num_q_heads, int32_t num_kv_heads, int32_t head_dim,
                             int32_t max_blocks_per_seq, int32_t chunk_size, int32_t total_q);

/* Zero the control words of a freshly allocated workspace (enqueued on `stream`).  Needed
 * once; every call leaves the workspace ready for the next.  Call it again after a call
 * reported a device-side error. */
int coopt_workspace_init(void* workspace, size_t workspace_bytes, void* stream);

/* Where a q_len == 1 coopt_paged_chunked call leaves its per-chunk partials: byte offsets
 * from `workspace` of o_c fp32 [batch][num_q_heads][max_chunks][head_dim] and of m_c and l_c,
 * both fp32 [batch][num_q_heads][max_chunks], max_chunks = ceil(max_blocks_per_seq * 16 /
 * chunk_size).  Host arithmetic only. */
int coopt_chunk_partials(int32_t batch, int32_t num_q_heads, int32_t head_dim, int32_t max_blocks_per_seq,
                         int32_t chunk_size, size_t* o_offset, size_t* m_offset, size_t* l_offset,
                         int32_t* max_chunks);

/*
 * coopt_selftest_bounded_wait -- diagnostic: one warp waits on a barrier that never completes, with the
 * same bounded wait every role of the attention kernels uses (a 2 s limit there), and gives up after
 * about limit_ns nanoseconds (1 .. 100,000,000).  The paper has no counterpart.  On return from the
 * stream, *status (DEVICE int32, zero before the call) holds COOPT_ERR_TIMEOUT and *elapsed_us (DEVICE
 * int32, may be NULL) the microseconds the warp waited; the context stays usable.
 * Errors: INVALID_ARG (null status, limit out of range), CUDA.
 */
int coopt_selftest_bounded_wait(uint64_t limit_ns, int32_t* status, int32_t* elapsed_us, void* stream);

const char* coopt_status_string(int status);
int coopt_version(void);

#ifdef __cplusplus
}
#endif
#endif /* COOPT_H_ */
