// What the Opt-KV write kernels and the fused decode step share: the scale rule of one (block, kv head,
// K | V) part (Algorithm 1 phase 1 with dynamic FP8 scales), token-group discovery, small helpers.
#pragma once

#include "coopt_common.cuh"

namespace coopt {

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
  if (lane == 0) g.n = 0;
  const int jb = i - 32 + lane, jf = i + lane;
  const int64_t sb = jb >= 0 ? p.slot_mapping[jb] : -1;
  const int64_t sf = jf < p.num_tokens ? p.slot_mapping[jf] : -1;
  const int64_t slot = __shfl_sync(0xffffffffu, sf, 0);
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

// Two fp32 values -> two E4M3 codes (lo in the low byte), round to nearest even, saturating.
__device__ __forceinline__ uint32_t f32x2_to_e4m3x2(float lo, float hi) {
  uint16_t d;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(d) : "f"(hi), "f"(lo));
  return d;
}

// Two fp32 values -> two E5M2 codes (lo in the low byte), round to nearest even, saturating.
__device__ __forceinline__ uint32_t f32x2_to_e5m2x2(float lo, float hi) {
  uint16_t d;
  asm("cvt.rn.satfinite.e5m2x2.f32 %0, %1, %2;" : "=h"(d) : "f"(hi), "f"(lo));
  return d;
}
template <bool kE5m2>
__device__ __forceinline__ uint32_t f32x2_to_codes(float lo, float hi) {
  return kE5m2 ? f32x2_to_e5m2x2(lo, hi) : f32x2_to_e4m3x2(lo, hi);
}

// kPerLane consecutive bf16 values of one row as packed pairs; one load when the row is aligned for it.
template <int kPerLane, bool kVec>
__device__ __forceinline__ void load_row(const __nv_bfloat16* row, uint32_t (&w)[kPerLane / 2]) {
  if constexpr (kVec) {
    if constexpr (kPerLane == 4) {
      const uint2 u = *reinterpret_cast<const uint2*>(row);
      w[0] = u.x; w[1] = u.y;
    } else {
      w[0] = *reinterpret_cast<const uint32_t*>(row);
    }
  } else {
    const unsigned short* r16 = reinterpret_cast<const unsigned short*>(row);
#pragma unroll
    for (int e = 0; e < kPerLane / 2; ++e) w[e] = static_cast<uint32_t>(r16[2 * e]) | (static_cast<uint32_t>(r16[2 * e + 1]) << 16);
  }
}
// element e of a row held as packed bf16 pairs, widened to fp32 (exact)
template <int kWords>
__device__ __forceinline__ float row_elem(const uint32_t (&w)[kWords], int e) {
  return __uint_as_float((e & 1) ? (w[e >> 1] & 0xffff0000u) : (w[e >> 1] << 16));
}

// One warp writes the K part (which = 0) or the V part (which = 1) of kv head h of the group's
// granule: it stages the part in shared memory (st, 16 * D bytes), applies the scale rule, and
// writes the part back with 16-byte stores.  A group that fills the whole block in order needs no
// resident codes; its V part goes from registers straight to memory.
// kTok bounds the group's size: 16 for the write kernels, 1 for the fused decode step (one new token per
// sequence); the arithmetic is the same instruction for instruction, so both give the same bytes.
// kE5m2 selects the code format (the E5M2 ablation): encoder, decoder and the format's largest value.
template <int D, int kTok = kBlockSize, bool kE5m2 = false>
__device__ __forceinline__ void write_part(const WriteParams& p, const Group& g, int h, int which, uint8_t* st, int lane) {
  constexpr int kPart = part_bytes(D, true);          // 16 * D bytes
  constexpr int kPerLane = D / 32;                    // dims handled by one lane
  const int n = g.n;
  bool fresh = false, full = (n == kBlockSize);
#pragma unroll
  for (int t = 0; t < kTok; ++t) {
    if (t < n) {
      fresh |= (g.off[t] == 0);
      full &= (g.off[t] == t);
    }
  }

  uint8_t* gran = p.cache + (static_cast<size_t>(g.blk) * p.num_kv_heads + h) * granule_bytes(D, true);
  float* scales = reinterpret_cast<float*>(gran + header_offset(D));
  const __nv_bfloat16* src = which == 0 ? p.k : p.v;
  uint8_t* part = gran + part_offset(D, true, which);
  uint4* st4 = reinterpret_cast<uint4*>(st);
  const bool vec = ((reinterpret_cast<uintptr_t>(src) | static_cast<uintptr_t>(p.token_stride * 2)) & (kPerLane * 2 - 1)) == 0;

  // every load of this part is issued before the first one is consumed: the old scale, the
  // resident codes (zeros for a block that is opened anew) and the group's rows.  Rows beyond
  // the group's size repeat its last row, so that no load waits on a branch.
  const float s_old = fresh ? 0.0f : scales[which];
  uint4 resident[kPart / 512];
#pragma unroll
  for (int c = 0; c < kPart / 512; ++c)
    resident[c] = (fresh || full) ? make_uint4(0, 0, 0, 0) : reinterpret_cast<const uint4*>(part)[c * 32 + lane];
  uint32_t raw[kTok][kPerLane / 2];
  const __nv_bfloat16* rows = src + h * D + lane * kPerLane;
  // a whole block of tokens that follow one another in the call (a bulk fill): no look-up of the rows
  const bool in_a_row = kTok > 1 && n == kTok && g.tok[kTok - 1] - g.tok[0] == kTok - 1;
  if (vec && in_a_row) {
    const __nv_bfloat16* r0 = rows + static_cast<int64_t>(g.tok[0]) * p.token_stride;
#pragma unroll
    for (int t = 0; t < kTok; ++t) load_row<kPerLane, true>(r0 + t * p.token_stride, raw[t]);
  } else if (vec) {
#pragma unroll
    for (int t = 0; t < kTok; ++t) load_row<kPerLane, true>(rows + static_cast<int64_t>(g.tok[min(t, n - 1)]) * p.token_stride, raw[t]);
  } else {
#pragma unroll
    for (int t = 0; t < kTok; ++t) load_row<kPerLane, false>(rows + static_cast<int64_t>(g.tok[min(t, n - 1)]) * p.token_stride, raw[t]);
  }
  if (!full) {
#pragma unroll
    for (int c = 0; c < kPart / 512; ++c) st4[c * 32 + lane] = resident[c];
  }
  // The largest magnitude, on the packed pairs: magnitudes of bf16 values order like their 15-bit patterns, and
  // the rows past the group's size repeat its last row, so no row has to be left out.
  uint32_t amax2 = 0;
#pragma unroll
  for (int t = 0; t < kTok; ++t)
#pragma unroll
    for (int e = 0; e < kPerLane / 2; ++e) amax2 = __vmaxu2(amax2, raw[t][e] & 0x7FFF7FFFu);
  float amax = __uint_as_float(max(amax2 << 16, amax2 & 0xFFFF0000u));
  amax = warp_max(amax);
  const float s_new = fmaxf(s_old, __fdiv_rn(amax, kE5m2 ? kE5m2Max : kE4m3Max));
  __syncwarp();

  // scale grew on a block that already holds tokens: re-express every resident code
  if (!fresh && s_new > s_old && s_old > 0.0f) {
    for (int i = lane; i < kPart; i += 32) {
      const float val = __fmul_rn(kE5m2 ? e5m2_to_f32(st[i]) : e4m3_to_f32(st[i]), s_old);
      st[i] = static_cast<uint8_t>(kE5m2 ? f32_to_e5m2(__fdiv_rn(val, s_new)) : f32_to_e4m3(__fdiv_rn(val, s_new)));
    }
    __syncwarp();
  }

  // x / s_new of element e of the group's t-th token (the value itself while the scale is zero).
  // One correctly rounded reciprocal serves the whole part: with r = RN(1 / s) and q0 = RN(x * r),
  // RN(q0 + (x - s * q0) * r) is the correctly rounded quotient as long as nothing under- or overflows.
  // |x| <= 448 * s here, and for s within 2^-40 .. 2^40 an underflow can only touch quotients far
  // below the smallest E4M3 magnitude, which encode to a signed zero either way; scales outside that
  // range take the division instruction.
  const bool by_rcp = s_new >= 0x1p-40f && s_new <= 0x1p40f;
  const float rcp = by_rcp ? __frcp_rn(s_new) : 0.0f;
  auto by_reciprocal = [&](int t, int e) -> float {
    const float xv = row_elem(raw[t], e);
    const float q0 = __fmul_rn(xv, rcp);
    return copysignf(__fmaf_rn(__fmaf_rn(-s_new, q0, xv), rcp, q0), xv);     // a zero keeps the sign of x
  };
  auto by_reciprocal_magnitude = [&](int t, int e) -> float {                // the same without the sign of a zero
    const float xv = row_elem(raw[t], e);
    const float q0 = __fmul_rn(xv, rcp);
    return __fmaf_rn(__fmaf_rn(-s_new, q0, xv), rcp, q0);
  };
  auto by_division = [&](int t, int e) -> float {
    const float xv = row_elem(raw[t], e);
    return s_new > 0.0f ? __fdiv_rn(xv, s_new) : xv;
  };

  auto encode = [&](auto scaled, auto scaled_k, bool k_signs_from_x) {
    if (kTok == kBlockSize && full && which == 1) {
      // V of a whole block: the 16 tokens of one dim are 16 consecutive bytes of the part
#pragma unroll
      for (int e = 0; e < kPerLane; ++e) {
        uint32_t w[4];
#pragma unroll
        for (int q = 0; q < 4; ++q)
          w[q] = f32x2_to_codes<kE5m2>(scaled((4 * q) % kTok, e), scaled((4 * q + 1) % kTok, e)) |
                 (f32x2_to_codes<kE5m2>(scaled((4 * q + 2) % kTok, e), scaled((4 * q + 3) % kTok, e)) << 16);
        *reinterpret_cast<uint4*>(part + v_elem_offset(D, true, 0, lane * kPerLane + e)) = make_uint4(w[0], w[1], w[2], w[3]);
      }
    } else {
      // encode the group's tokens into their permuted places
#pragma unroll
      for (int t = 0; t < kTok; ++t) {
        if (t < n) {
          const int off = g.off[t];
          if (which == 0) {
            // the lane's dims are consecutive bytes of a K row
            uint8_t* dst = st + k_elem_offset(D, true, off, lane * kPerLane);
            if constexpr (kPerLane == 4) {
              // four codes of one token; the signs (which a zero quotient may have lost) are those of the four
              // values themselves: the top bits of the upper bytes of the packed pairs, gathered in one go
              uint32_t word = f32x2_to_codes<kE5m2>(scaled_k(t, 0), scaled_k(t, 1)) | (f32x2_to_codes<kE5m2>(scaled_k(t, 2), scaled_k(t, 3)) << 16);
              if (k_signs_from_x) word |= __byte_perm(raw[t][0], raw[t][1], 0x7531) & 0x80808080u;
              *reinterpret_cast<uint32_t*>(dst) = word;
            } else
              *reinterpret_cast<uint16_t*>(dst) = static_cast<uint16_t>(f32x2_to_codes<kE5m2>(scaled(t, 0), scaled(t, 1)));
          } else {
#pragma unroll
            for (int e = 0; e < kPerLane; ++e)
              st[v_elem_offset(D, true, off, lane * kPerLane + e)] = static_cast<uint8_t>(kE5m2 ? f32_to_e5m2(scaled(t, e)) : f32_to_e4m3(scaled(t, e)));
          }
        }
      }
      __syncwarp();
      uint4* out4 = reinterpret_cast<uint4*>(part);
#pragma unroll
      for (int c = 0; c < kPart / 512; ++c) out4[c * 32 + lane] = st4[c * 32 + lane];
    }
  };
  if (by_rcp) encode(by_reciprocal, by_reciprocal_magnitude, true); else encode(by_division, by_division, false);
  if (lane == 0) scales[which] = s_new;
  if (which == 0 && fresh && lane < 6) scales[2 + lane] = 0.0f;       // rest of the header
  __syncwarp();
}

}  // namespace coopt
