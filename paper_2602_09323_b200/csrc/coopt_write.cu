// coopt_kv_write: Opt-KV cache write (Algorithm 1 phase 1, Eq. 5) with per-(block, kv head)
// dynamic FP8 E4M3 scales.  One warp owns one (token group, kv head): it is the only writer of
// that granule during the call, so the scale update and the re-expression of resident codes
// need no atomics.
#include "coopt_common.cuh"

namespace coopt {

namespace {

constexpr int kWriteHeads = 4;                 // kv heads per CTA
constexpr int kWriteWarps = 2 * kWriteHeads;   // FP8: one warp per (kv head, K | V)

struct WriteParams {
  uint8_t* cache;
  const __nv_bfloat16* k;
  const __nv_bfloat16* v;
  const int64_t* slot_mapping;
  int64_t token_stride;
  int num_tokens;
  int num_kv_heads;
  int num_blocks;
};

__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
  return x;
}

// Token group discovery, identical for every warp of the CTA (uniform control flow).
// The group leader is the first non-skipped token of a run of non-skipped tokens that share a
// block; skipped tokens (slot < 0, Eq. 5) inside the run are stepped over.
struct Group {
  int n;        // tokens in the group (0 = this CTA has nothing to do)
  int blk;
  int tok[kBlockSize];
  int off[kBlockSize];
};

__device__ __forceinline__ void find_group(const WriteParams& p, int i, Group& g) {
  g.n = 0;
  const int64_t slot = p.slot_mapping[i];
  if (slot < 0) return;                                   // Eq. 5: skipped token
  const int64_t blk = slot / kBlockSize;
  if (blk >= p.num_blocks) return;
  int prev = i - 1;
  while (prev >= 0 && p.slot_mapping[prev] < 0) --prev;
  if (prev >= 0 && p.slot_mapping[prev] / kBlockSize == blk) return;   // not the leader
  g.blk = static_cast<int>(blk);
  for (int t = i; t < p.num_tokens && g.n < kBlockSize; ++t) {
    const int64_t s = p.slot_mapping[t];
    if (s < 0) continue;
    if (s / kBlockSize != blk) break;
    g.tok[g.n] = t;
    g.off[g.n] = static_cast<int>(s % kBlockSize);
    ++g.n;
  }
}

// The same discovery by one warp in a single trip to memory: 32 slots before token i and 32 from it
// on are looked at together.  Neighbourhoods that the two windows do not settle (long runs of skipped
// tokens) fall back to the serial walk.
__device__ __forceinline__ void find_group_warp(const WriteParams& p, int i, Group& g, int lane) {
  const int jb = i - 32 + lane, jf = i + lane;
  const int64_t sb = jb >= 0 ? p.slot_mapping[jb] : -1;
  const int64_t sf = jf < p.num_tokens ? p.slot_mapping[jf] : -1;
  const int64_t slot = __shfl_sync(0xffffffffu, sf, 0);
  if (lane == 0) g.n = 0;
  if (slot < 0) return;                                   // Eq. 5: skipped token
  const int64_t blk = slot / kBlockSize;
  if (blk >= p.num_blocks) return;
  const unsigned before = __ballot_sync(0xffffffffu, sb >= 0);
  const unsigned same = __ballot_sync(0xffffffffu, sf >= 0 && sf / kBlockSize == blk);
  const unsigned other = __ballot_sync(0xffffffffu, sf >= 0 && sf / kBlockSize != blk);
  const unsigned mem = same & (other ? (1u << (__ffs(other) - 1)) - 1u : 0xffffffffu);
  const bool back_known = before != 0 || i <= 32;
  const bool fwd_known = other != 0 || i + 32 >= p.num_tokens || __popc(mem) >= kBlockSize;
  if (!back_known || !fwd_known) {
    if (lane == 0) find_group(p, i, g);
    return;
  }
  if (before != 0) {
    const int64_t sp = __shfl_sync(0xffffffffu, sb, 31 - __clz(before));
    if (sp / kBlockSize == blk) return;                   // not the leader of its group
  }
  const int rank = __popc(mem & ((1u << lane) - 1u));
  if (((mem >> lane) & 1u) && rank < kBlockSize) {
    g.tok[rank] = jf;
    g.off[rank] = static_cast<int>(sf % kBlockSize);
  }
  if (lane == 0) {
    g.blk = static_cast<int>(blk);
    g.n = min(__popc(mem), kBlockSize);
  }
}

// FP8 path.  One warp per (kv head, K | V): it stages that part of its granule in shared memory,
// applies the scale rule, and writes the part back with 16-byte stores.
template <int D>
__global__ void __launch_bounds__(kWriteWarps * 32) kv_write_fp8_kernel(WriteParams p) {
  constexpr int kPart = part_bytes(D, true);          // 16 * D bytes
  constexpr int kPerLane = D / 32;                    // dims handled by one lane
  __shared__ __align__(16) uint8_t stage[kWriteWarps][kPart];
  __shared__ Group group;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (warp == 0) find_group_warp(p, blockIdx.x, group, lane);
  __syncthreads();
  const int n = group.n;
  if (n == 0) return;
  const int h = blockIdx.y * kWriteHeads + (warp >> 1);
  const int which = warp & 1;
  if (h >= p.num_kv_heads) return;

  bool fresh = false;
  for (int t = 0; t < n; ++t) fresh |= (group.off[t] == 0);

  uint8_t* gran = p.cache + (static_cast<size_t>(group.blk) * p.num_kv_heads + h) * granule_bytes(D, true);
  float* scales = reinterpret_cast<float*>(gran + header_offset(D));
  uint8_t* st = stage[warp];

  {
    const __nv_bfloat16* src = which == 0 ? p.k : p.v;
    uint8_t* part = gran + part_offset(D, true, which);

    // resident codes (or zeros for a block that is opened anew)
    uint4* st4 = reinterpret_cast<uint4*>(st);
    const uint4* part4 = reinterpret_cast<const uint4*>(part);
#pragma unroll
    for (int c = 0; c < kPart / 512; ++c)
      st4[c * 32 + lane] = fresh ? make_uint4(0, 0, 0, 0) : part4[c * 32 + lane];

    // new values and their amax
    float x[kBlockSize][kPerLane];
    float amax = 0.0f;
#pragma unroll
    for (int t = 0; t < kBlockSize; ++t) {
      if (t < n) {
        const __nv_bfloat16* row = src + static_cast<int64_t>(group.tok[t]) * p.token_stride + h * D + lane * kPerLane;
#pragma unroll
        for (int e = 0; e < kPerLane; ++e) {
          x[t][e] = __bfloat162float(row[e]);
          amax = fmaxf(amax, fabsf(x[t][e]));
        }
      }
    }
    amax = warp_max(amax);
    const float s_old = fresh ? 0.0f : scales[which];
    const float s_new = fmaxf(s_old, __fdiv_rn(amax, kE4m3Max));
    __syncwarp();

    // scale grew on a block that already holds tokens: re-express every resident code
    if (!fresh && s_new > s_old && s_old > 0.0f) {
      for (int i = lane; i < kPart; i += 32) {
        const float val = __fmul_rn(e4m3_to_f32(st[i]), s_old);
        st[i] = static_cast<uint8_t>(f32_to_e4m3(__fdiv_rn(val, s_new)));
      }
      __syncwarp();
    }

    // encode the group's tokens into their permuted places
#pragma unroll
    for (int t = 0; t < kBlockSize; ++t) {
      if (t < n) {
        const int off = group.off[t];
#pragma unroll
        for (int e = 0; e < kPerLane; ++e) {
          const int d = lane * kPerLane + e;
          const float y = s_new > 0.0f ? __fdiv_rn(x[t][e], s_new) : x[t][e];
          const int pos = which == 0 ? k_elem_offset(D, true, off, d) : v_elem_offset(D, true, off, d);
          st[pos] = static_cast<uint8_t>(f32_to_e4m3(y));
        }
      }
    }
    __syncwarp();

    uint4* out4 = reinterpret_cast<uint4*>(part);
#pragma unroll
    for (int c = 0; c < kPart / 512; ++c) out4[c * 32 + lane] = st4[c * 32 + lane];
    if (lane == 0) scales[which] = s_new;
    __syncwarp();
  }
  if (which == 0 && fresh && lane < 6) scales[2 + lane] = 0.0f;       // rest of the header
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
  const bool fp8 = c->dtype == COOPT_KV_FP8_E4M3;
  // FP8: a CTA serves kWriteHeads kv heads (two warps each); bf16: kWriteWarps heads (one warp each)
  const int heads_per_cta = fp8 ? kWriteHeads : kWriteWarps;
  const dim3 grid(num_tokens, (c->num_kv_heads + heads_per_cta - 1) / heads_per_cta);
  if (c->head_dim == 128) {
    if (fp8) kv_write_fp8_kernel<128><<<grid, block, 0, stream>>>(p);
    else kv_write_bf16_kernel<128><<<grid, block, 0, stream>>>(p);
  } else {
    if (fp8) kv_write_fp8_kernel<64><<<grid, block, 0, stream>>>(p);
    else kv_write_bf16_kernel<64><<<grid, block, 0, stream>>>(p);
  }
  return cudaGetLastError() == cudaSuccess ? COOPT_OK : COOPT_ERR_CUDA;
}

}  // namespace coopt
