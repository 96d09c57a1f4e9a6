// coopt_kv_write: Opt-KV cache write (Algorithm 1 phase 1, Eq. 5) with per-(block, kv head)
// dynamic FP8 E4M3 scales.  One warp owns one (token group, kv head): it is the only writer of
// that granule during the call, so the scale update and the re-expression of resident codes
// need no atomics.
#include "coopt_write.cuh"

namespace coopt {

namespace {

constexpr int kWriteHeads = 4;                 // kv heads per CTA
constexpr int kWriteWarps = 2 * kWriteHeads;   // FP8: one warp per (kv head, K | V)

// FP8, few tokens (decode steps): one CTA per (token, kWriteHeads kv heads), one warp per
// (kv head, K | V); CTAs whose token leads no group leave at once.
template <int D, bool kE5m2>
__global__ void __launch_bounds__(kWriteWarps * 32) kv_write_fp8_kernel(WriteParams p) {
  __shared__ __align__(16) uint8_t stage[kWriteWarps][part_bytes(D, true)];
  __shared__ Group group;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (warp == 0) find_group_warp(p, blockIdx.x, group, lane);
  __syncthreads();
  if (group.n == 0) return;
  const int h = blockIdx.y * kWriteHeads + (warp >> 1);
  if (h >= p.num_kv_heads) return;
  write_part<D, kBlockSize, kE5m2>(p, group, h, warp & 1, stage[warp], lane);
}

// FP8, many tokens (prefill chunks, bulk fills): one CTA per (kSpan consecutive tokens, kWriteHeads
// kv heads).  Every warp settles one token of the span in the same memory trip; the groups found
// (one per 16 tokens in a contiguous fill) are then served by all warps.
constexpr int kSpan = 4 * kWriteWarps;  // a contiguous fill starts a group every 16 tokens: every CTA finds one
constexpr int kSpanThreshold = 512;     // calls with more tokens than this take the span kernel
template <int D, bool kE5m2>
__global__ void __launch_bounds__(kWriteWarps * 32, 3) kv_write_fp8_span_kernel(WriteParams p) {
  __shared__ __align__(16) uint8_t stage[kWriteWarps][part_bytes(D, true)];
  __shared__ Group groups[kSpan];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int w = warp; w < kSpan; w += kWriteWarps) {
    const int tok = blockIdx.x * kSpan + w;
    if (tok < p.num_tokens) find_group_warp(p, tok, groups[w], lane);
    else if (lane == 0) groups[w].n = 0;
  }
  __syncthreads();
  unsigned leaders = 0;
#pragma unroll
  for (int w = 0; w < kSpan; ++w) leaders |= (groups[w].n > 0 ? 1u : 0u) << w;
  const int h = blockIdx.y * kWriteHeads + (warp >> 1);
  if (h >= p.num_kv_heads) return;
  while (leaders) {
    const int w = __ffs(leaders) - 1;
    leaders &= leaders - 1;
    write_part<D, kBlockSize, kE5m2>(p, groups[w], h, warp & 1, stage[warp], lane);
  }
}

// bf16 ablation cache: store the values unchanged at their permuted places.
template <int D>
__global__ void __launch_bounds__(kWriteWarps * 32) kv_write_bf16_kernel(WriteParams p) {
  constexpr int kPerLane = D / 32;
  const int i = blockIdx.x;
  const int64_t slot = p.slot_mapping[i];
  if (slot < 0) return;                                   // Eq. 5
  const int64_t blk = slot / kBlockSize;
  if (blk >= p.num_blocks) return;
  const int off = static_cast<int>(slot % kBlockSize);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int h = blockIdx.y * kWriteWarps + warp;
  if (h >= p.num_kv_heads) return;
  uint8_t* gran = p.cache + (static_cast<size_t>(blk) * p.num_kv_heads + h) * granule_bytes(D, false);
#pragma unroll
  for (int which = 0; which < 2; ++which) {
    const __nv_bfloat16* row = (which == 0 ? p.k : p.v) + static_cast<int64_t>(i) * p.token_stride + h * D + lane * kPerLane;
    uint8_t* part = gran + part_offset(D, false, which);
#pragma unroll
    for (int e = 0; e < kPerLane; ++e) {
      const int d = lane * kPerLane + e;
      const int pos = which == 0 ? k_elem_offset(D, false, off, d) : v_elem_offset(D, false, off, d);
      *reinterpret_cast<__nv_bfloat16*>(part + pos) = row[e];
    }
  }
}

}  // namespace

int launch_kv_write(const coopt_cache* c, const void* k, const void* v, int64_t stride, const int64_t* slots,
                    int num_tokens, cudaStream_t stream) {
  WriteParams p;
  p.cache = static_cast<uint8_t*>(c->data);
  p.k = static_cast<const __nv_bfloat16*>(k);
  p.v = static_cast<const __nv_bfloat16*>(v);
  p.slot_mapping = slots;
  p.token_stride = stride;
  p.num_tokens = num_tokens;
  p.num_kv_heads = c->num_kv_heads;
  p.num_blocks = c->num_blocks;
  const dim3 block(kWriteWarps * 32);
  const bool fp8 = is_fp8(c->dtype), e5m2 = c->dtype == COOPT_KV_FP8_E5M2;
  // FP8: a CTA serves kWriteHeads kv heads (two warps each); bf16: kWriteWarps heads (one warp each)
  const int heads_per_cta = fp8 ? kWriteHeads : kWriteWarps;
  const int head_ctas = (c->num_kv_heads + heads_per_cta - 1) / heads_per_cta;
  const dim3 grid(num_tokens, head_ctas);
  const dim3 span_grid((num_tokens + kSpan - 1) / kSpan, head_ctas);
  const bool span = fp8 && num_tokens > kSpanThreshold;
  if (c->head_dim == 128) {
    if (span && e5m2) kv_write_fp8_span_kernel<128, true><<<span_grid, block, 0, stream>>>(p);
    else if (span) kv_write_fp8_span_kernel<128, false><<<span_grid, block, 0, stream>>>(p);
    else if (e5m2) kv_write_fp8_kernel<128, true><<<grid, block, 0, stream>>>(p);
    else if (fp8) kv_write_fp8_kernel<128, false><<<grid, block, 0, stream>>>(p);
    else kv_write_bf16_kernel<128><<<grid, block, 0, stream>>>(p);
  } else {
    if (span && e5m2) kv_write_fp8_span_kernel<64, true><<<span_grid, block, 0, stream>>>(p);
    else if (span) kv_write_fp8_span_kernel<64, false><<<span_grid, block, 0, stream>>>(p);
    else if (e5m2) kv_write_fp8_kernel<64, true><<<grid, block, 0, stream>>>(p);
    else if (fp8) kv_write_fp8_kernel<64, false><<<grid, block, 0, stream>>>(p);
    else kv_write_bf16_kernel<64><<<grid, block, 0, stream>>>(p);
  }
  return cudaGetLastError() == cudaSuccess ? COOPT_OK : COOPT_ERR_CUDA;
}

}  // namespace coopt
