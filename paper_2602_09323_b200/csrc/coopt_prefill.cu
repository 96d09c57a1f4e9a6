// Chunked prefill against the paged FP8 cache: Eq. 1 with the causal K_{<=t}, Eq. 6
// dequantisation on load, Eq. 7-8 grouped-query sharing, Eq. 9 valid blocks only, Eq. 10
// max-subtracted softmax, for runs of several query tokens per sequence.
//
// A CTA owns one (sequence, kv head, tile of consecutive query tokens).  Its 128 rows are the
// (query token, query head of the group) pairs of the tile, so the K/V stream of the kv head is
// fetched once for all G heads (Algorithm 2).  The context is walked 64 tokens (four cache
// blocks) at a time:
//   1. one lane per block starts a bulk async copy of the granule into a ring of raw stages
//      (an mbarrier per stage counts the bytes);
//   2. all threads widen the E4M3 codes of the stage to f16 (exact) into a double-buffered
//      operand tile laid out in the register order of the matrix instruction;
//   3. every warp runs S = Q K^T and O += P V for its 16 rows on tensor cores
//      (mma.sync m16n8k16, f16 operands, fp32 accumulators) with an online softmax in between.
// The K scale of a block is applied to the logits of its 16 tokens and the V scale is folded
// into the probabilities, both uniform per block, so the products themselves are exact.
#include "coopt_common.cuh"

namespace coopt {

namespace {

constexpr int kPfWarps = 8;
constexpr int kPfThreads = kPfWarps * 32;
constexpr int kPfRows = kPfWarps * 16;
constexpr int kTileBlocks = 4;                         // cache blocks per tile
constexpr int kTileTokens = kTileBlocks * kBlockSize;  // 64
constexpr int kRawStages = 3;
constexpr float kLog2e = 1.4426950408889634f;

struct PrefillParams {
  const uint8_t* cache;
  const __nv_bfloat16* q;
  __nv_bfloat16* out;
  const int* cu_q_lens;
  const int* block_table;
  const int* context_lens;
  int max_blocks_per_seq;
  int batch, num_q_heads, num_kv_heads, group;
  int num_blocks;
  int tile_queries;        // query tokens per CTA = 128 / group
  int causal;
  float sm_scale_log2;
  int* status;
};

template <int D>
struct PfCfg {
  static constexpr int kGran = granule_bytes(D, true);
  static constexpr int kRawStage = kTileBlocks * kGran;
  static constexpr int kConvBlock = 2 * (2 * kBlockSize * D);   // f16 K and V of one block
  static constexpr int kConvTile = kTileBlocks * kConvBlock;
  static constexpr int kChunksPerBlock = 2 * D;                 // 16-byte chunks of codes (K then V)
  static constexpr int kRawOff = 0;
  static constexpr int kConvOff = kRawOff + kRawStages * kRawStage;
  static constexpr int kScaleOff = kConvOff + 2 * kConvTile;    // float [2 buffers][4 blocks][2]
  static constexpr int kBarOff = kScaleOff + 2 * kTileBlocks * 2 * 4;
  static constexpr int kMiscOff = kBarOff + kRawStages * 8;
  static constexpr int kSmemBytes = kMiscOff + 32;
};

__device__ __forceinline__ float quad_max(float x) {
  x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 1));
  return fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 2));
}
__device__ __forceinline__ float quad_sum(float x) {
  x += __shfl_xor_sync(0xffffffffu, x, 1);
  return x + __shfl_xor_sync(0xffffffffu, x, 2);
}
template <int D>
__global__ void __launch_bounds__(kPfThreads, 1) paged_prefill_kernel(const PrefillParams p) {
  using C = PfCfg<D>;
  constexpr int kKSteps = D / 16, kNTiles = D / 8;
  extern __shared__ __align__(128) uint8_t smem[];
  uint8_t* raw = smem + C::kRawOff;
  uint8_t* conv = smem + C::kConvOff;
  float* tile_scales = reinterpret_cast<float*>(smem + C::kScaleOff);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::kBarOff);
  int* misc = reinterpret_cast<int*>(smem + C::kMiscOff);   // [0] sequence, [1] first query of the tile

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int quad = lane & 3;
  const int G = p.group, Hq = p.num_q_heads, Hkv = p.num_kv_heads;
  const int g = blockIdx.y;
  const int TQ = p.tile_queries;

  // ---- which (sequence, query tile) is this CTA's ----------------------------------------------
  if (tid == 0) {
    int left = blockIdx.x, found = -1, q0 = 0;
    for (int b = 0; b < p.batch; ++b) {
      const int n = max(0, p.cu_q_lens[b + 1] - p.cu_q_lens[b]);
      const int nt = (n + TQ - 1) / TQ;
      if (left < nt) { found = b; q0 = (nt - 1 - left) * TQ; break; }   // late (long) tiles first
      left -= nt;
    }
    misc[0] = found;
    misc[1] = q0;
    for (int i = 0; i < kRawStages; ++i) mbar_init(&bars[i], 1);
    mbar_fence_init();
  }
  __syncthreads();
  const int b = misc[0];
  if (b < 0) return;
  const int q0 = misc[1];
  const int row_base = p.cu_q_lens[b];
  const int n_new = p.cu_q_lens[b + 1] - row_base;
  const int nq = min(TQ, n_new - q0);
  const int L = max(0, min(p.context_lens[b], p.max_blocks_per_seq * kBlockSize));
  // last position any row of the tile may see (Eq. 1: K_{<=t})
  const int kv_end = p.causal ? max(0, min(L, L - n_new + q0 + nq)) : L;
  const int n_tiles = (kv_end + kTileTokens - 1) / kTileTokens;
  const int n_blocks = (kv_end + kBlockSize - 1) / kBlockSize;

  // ---- the two rows of this lane ------------------------------------------------------------------
  const int r0 = warp * 16 + (lane >> 2), r1 = r0 + 8;
  const int qi0 = r0 / G, qi1 = r1 / G;
  const bool live0 = qi0 < nq, live1 = qi1 < nq;
  const size_t grow0 = static_cast<size_t>(row_base + q0 + (live0 ? qi0 : 0)) * Hq + g * G + (live0 ? r0 % G : 0);
  const size_t grow1 = static_cast<size_t>(row_base + q0 + (live1 ? qi1 : 0)) * Hq + g * G + (live1 ? r1 % G : 0);
  // index of the last visible token of each row; -1 hides everything
  int lim0 = -1, lim1 = -1;
  if (live0) lim0 = p.causal ? min(L - 1, L - n_new + q0 + qi0) : L - 1;
  if (live1) lim1 = p.causal ? min(L - 1, L - n_new + q0 + qi1) : L - 1;
  int warp_min_lim = min(lim0, lim1);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) warp_min_lim = min(warp_min_lim, __shfl_xor_sync(0xffffffffu, warp_min_lim, o));

  // ---- producer state (warp 0, lanes 0..3: one cache block each) --------------------------------
  const int* trow = p.block_table + static_cast<size_t>(b) * p.max_blocks_per_seq;
  int issued = 0;
  int next_id = 0;
  auto load_id = [&](int tile) {
    const int j = tile * kTileBlocks + lane;
    if (warp == 0 && lane < kTileBlocks && j < n_blocks) {
      int id = trow[j];
      if (id < 0 || id >= p.num_blocks) { atomicCAS(p.status, 0, COOPT_ERR_INVALID_ARG); id = 0; }
      next_id = id;
    }
  };
  auto issue = [&]() {   // warp 0 only: copies of tile `issued` into its ring stage
    const int tile = issued;
    const int stage = tile % kRawStages;
    const int nb = min(kTileBlocks, n_blocks - tile * kTileBlocks);
    if (lane == 0) {
      fence_proxy_async();
      mbar_expect_tx(&bars[stage], nb * C::kGran);
    }
    __syncwarp();
    if (lane < nb) {
      const uint8_t* src = p.cache + (static_cast<size_t>(next_id) * Hkv + g) * C::kGran;
      bulk_copy_g2s(raw + stage * C::kRawStage + lane * C::kGran, src, C::kGran, &bars[stage]);
    }
    load_id(tile + 1);
  };
  if (warp == 0) load_id(0);
  for (int s = 0; s < kRawStages && s < n_tiles; ++s) {
    if (warp == 0) issue();
    ++issued;
  }

  // ---- query fragments: bf16 -> f16 after an exact power-of-two scaling per row ----------------
  uint32_t qa[kKSteps][4];
  float qs0 = p.sm_scale_log2, qs1 = p.sm_scale_log2;
  {
    uint32_t w0[kKSteps][2], w1[kKSteps][2];
    // k-step s of the instruction covers dims 16s..16s+15; its logical k positions 2c, 2c+1 (registers
    // a0/a1 and b0) stand for dims 16s + 4c + {0, 1}, positions 2c+8, 2c+9 (a2/a3 and b1) for dims
    // 16s + 4c + {2, 3}: the order in which a 16-byte chunk of the cache's K part splits over a quad
    const __nv_bfloat16* qp0 = p.q + grow0 * D + 4 * quad;
    const __nv_bfloat16* qp1 = p.q + grow1 * D + 4 * quad;
    float am0 = 0.0f, am1 = 0.0f;
#pragma unroll
    for (int s = 0; s < kKSteps; ++s)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        w0[s][e] = live0 ? *reinterpret_cast<const uint32_t*>(qp0 + 16 * s + 2 * e) : 0u;
        w1[s][e] = live1 ? *reinterpret_cast<const uint32_t*>(qp1 + 16 * s + 2 * e) : 0u;
        am0 = fmaxf(am0, fmaxf(fabsf(bf16_lo(w0[s][e])), fabsf(bf16_hi(w0[s][e]))));
        am1 = fmaxf(am1, fmaxf(fabsf(bf16_lo(w1[s][e])), fabsf(bf16_hi(w1[s][e]))));
      }
    am0 = quad_max(am0);
    am1 = quad_max(am1);
    auto pow2 = [](float amax, float& up, float& down) {
      int k2 = 0;
      if (amax > 0.0f) k2 = max(-64, min(64, 134 - static_cast<int>((__float_as_uint(amax) >> 23) & 0xFF)));
      up = __uint_as_float(static_cast<uint32_t>(k2 + 127) << 23);
      down = __uint_as_float(static_cast<uint32_t>(127 - k2) << 23);
    };
    float up0, dn0, up1, dn1;
    pow2(am0, up0, dn0);
    pow2(am1, up1, dn1);
    qs0 *= dn0;
    qs1 *= dn1;
#pragma unroll
    for (int s = 0; s < kKSteps; ++s) {
      qa[s][0] = pack_f16x2(bf16_lo(w0[s][0]) * up0, bf16_hi(w0[s][0]) * up0);
      qa[s][1] = pack_f16x2(bf16_lo(w1[s][0]) * up1, bf16_hi(w1[s][0]) * up1);
      qa[s][2] = pack_f16x2(bf16_lo(w0[s][1]) * up0, bf16_hi(w0[s][1]) * up0);
      qa[s][3] = pack_f16x2(bf16_lo(w1[s][1]) * up1, bf16_hi(w1[s][1]) * up1);
    }
  }

  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.0f, l1 = 0.0f, vref = 0.0f;
  float o[kNTiles][4];
#pragma unroll
  for (int t = 0; t < kNTiles; ++t)
#pragma unroll
    for (int e = 0; e < 4; ++e) o[t][e] = 0.0f;

  bool failed = false;
#pragma unroll 1
  for (int tile = 0; tile < n_tiles; ++tile) {
    const int stage = tile % kRawStages;
    const uint32_t parity = (tile / kRawStages) & 1u;
    const bool ok = mbar_wait_bounded(&bars[stage], parity);
    const int buf = tile & 1;
    uint8_t* cv = conv + buf * C::kConvTile;
    const int nb = min(kTileBlocks, n_blocks - tile * kTileBlocks);

    // ---- widen the stage's codes to f16 and put them in the register order of mma.m16n8k16 --------
    // A 16-byte chunk of the K part is one token x 16 dims, of the V part one dim x 16 tokens; either
    // way it feeds the four lanes of one quad with two registers each.
    if (ok) {
      const uint8_t* rs = raw + stage * C::kRawStage;
#pragma unroll
      for (int c = tid; c < kTileBlocks * C::kChunksPerBlock; c += kPfThreads) {
        const int jb = c / C::kChunksPerBlock, cc = c % C::kChunksPerBlock;
        uint4 w = make_uint4(0u, 0u, 0u, 0u);
        if (jb < nb) w = lds128(rs + jb * C::kGran + cc * 16);
        uint8_t* dst;
        uint32_t b0[4], b1[4];
        if (cc < D) {
          const int rg = cc / (D / 2), rem = cc % (D / 2), u = rem >> 3, n = rem & 7;   // token 8 rg + n, dims 16u..16u+15
          dst = cv + jb * C::kConvBlock + (rg * (D / 64) + (u >> 2)) * 1024 + ((u & 3) >> 1) * 512 + (4 * n) * 16 + (u & 1) * 8;
          const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
          for (int q = 0; q < 4; ++q) { b0[q] = e4m3x2_to_f16x2_lo(ww[q]); b1[q] = e4m3x2_to_f16x2_hi(ww[q]); }
        } else {
          const int d = cc - D, j = d >> 3, n = d & 7;                                  // dim d, tokens 0..15
          const int tok0 = (tile * kTileBlocks + jb) * kBlockSize;
          if (jb < nb && tok0 + kBlockSize > L) {
            // V codes of slots past the context are cleared so that stale bytes cannot reach P V
            const int keep = L - tok0;
            uint32_t* wm = reinterpret_cast<uint32_t*>(&w);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const int left = keep - 4 * q;
              wm[q] &= left >= 4 ? 0xFFFFFFFFu : (left <= 0 ? 0u : (1u << (8 * left)) - 1u);
            }
          }
          dst = cv + jb * C::kConvBlock + (D / 32) * 1024 + (j >> 2) * 1024 + ((j & 3) >> 1) * 512 + (4 * n) * 16 + (j & 1) * 8;
          // lane c of the quad: b0 = tokens 2c, 2c+1, b1 = tokens 2c+8, 2c+9
          b0[0] = e4m3x2_to_f16x2_lo(w.x); b0[1] = e4m3x2_to_f16x2_hi(w.x); b0[2] = e4m3x2_to_f16x2_lo(w.y); b0[3] = e4m3x2_to_f16x2_hi(w.y);
          b1[0] = e4m3x2_to_f16x2_lo(w.z); b1[1] = e4m3x2_to_f16x2_hi(w.z); b1[2] = e4m3x2_to_f16x2_lo(w.w); b1[3] = e4m3x2_to_f16x2_hi(w.w);
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) *reinterpret_cast<uint2*>(dst + q * 16) = make_uint2(b0[q], b1[q]);
      }
      if (tid < kTileBlocks * 2) {
        const int jb = tid >> 1;
        tile_scales[buf * kTileBlocks * 2 + tid] =
            jb < nb ? reinterpret_cast<const float*>(rs + jb * C::kGran + header_offset(D))[tid & 1] : 0.0f;
      }
    }
    // operand tile complete, raw stage free again; a wait that ran out ends the walk for everyone
    if (__syncthreads_or(!ok)) {
      failed = true;
      break;
    }
    if (issued < n_tiles) {
      if (warp == 0) issue();
      ++issued;
    }

    // ---- S = Q K^T: 16 rows x 64 tokens ------------------------------------------------------------
    float s[2 * kTileBlocks][4];
#pragma unroll
    for (int j = 0; j < 2 * kTileBlocks; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) s[j][e] = 0.0f;
#pragma unroll
    for (int jb = 0; jb < kTileBlocks; ++jb) {
      const uint8_t* kp = cv + jb * C::kConvBlock + lane * 16;
#pragma unroll
      for (int nt = 0; nt < 2; ++nt)
#pragma unroll
        for (int i = 0; i < D / 64; ++i) {
          const uint4 a = lds128(kp + (nt * (D / 64) + i) * 1024);
          const uint4 c = lds128(kp + (nt * (D / 64) + i) * 1024 + 512);
          mma16816<true>(s[2 * jb + nt], qa[4 * i][0], qa[4 * i][1], qa[4 * i][2], qa[4 * i][3], a.x, a.y);
          mma16816<true>(s[2 * jb + nt], qa[4 * i + 1][0], qa[4 * i + 1][1], qa[4 * i + 1][2], qa[4 * i + 1][3], a.z, a.w);
          mma16816<true>(s[2 * jb + nt], qa[4 * i + 2][0], qa[4 * i + 2][1], qa[4 * i + 2][2], qa[4 * i + 2][3], c.x, c.y);
          mma16816<true>(s[2 * jb + nt], qa[4 * i + 3][0], qa[4 * i + 3][1], qa[4 * i + 3][2], qa[4 * i + 3][3], c.z, c.w);
        }
    }

    // ---- logits in log2 units, causal / tail mask, online softmax (Eq. 10) -----------------------
    const float* ts = tile_scales + buf * kTileBlocks * 2;
    float vmax = 0.0f;
#pragma unroll
    for (int jb = 0; jb < kTileBlocks; ++jb) {
      const float sk = ts[2 * jb];
      vmax = fmaxf(vmax, ts[2 * jb + 1]);
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        s[2 * jb + nt][0] *= qs0 * sk; s[2 * jb + nt][1] *= qs0 * sk;
        s[2 * jb + nt][2] *= qs1 * sk; s[2 * jb + nt][3] *= qs1 * sk;
      }
    }
    const int tok_base = tile * kTileTokens;
    if (tok_base + kTileTokens - 1 > warp_min_lim) {
#pragma unroll
      for (int j = 0; j < 2 * kTileBlocks; ++j) {
        const int t0 = tok_base + 8 * j + 2 * quad;
        s[j][0] = t0 <= lim0 ? s[j][0] : -INFINITY;
        s[j][1] = t0 + 1 <= lim0 ? s[j][1] : -INFINITY;
        s[j][2] = t0 <= lim1 ? s[j][2] : -INFINITY;
        s[j][3] = t0 + 1 <= lim1 ? s[j][3] : -INFINITY;
      }
    }
    float mt0 = -INFINITY, mt1 = -INFINITY;
#pragma unroll
    for (int j = 0; j < 2 * kTileBlocks; ++j) {
      mt0 = fmaxf(mt0, fmaxf(s[j][0], s[j][1]));
      mt1 = fmaxf(mt1, fmaxf(s[j][2], s[j][3]));
    }
    const float mn0 = fmaxf(m0, quad_max(mt0)), mn1 = fmaxf(m1, quad_max(mt1));
    const float mu0 = mn0 == -INFINITY ? 0.0f : mn0, mu1 = mn1 == -INFINITY ? 0.0f : mn1;
    const float am0 = ex2(m0 - mu0), am1 = ex2(m1 - mu1);
    m0 = mn0;
    m1 = mn1;
    // o holds sum p * (sV / vref) * codes with vref the largest V scale met so far
    const float vnew = fmaxf(vref, vmax);
    const float vr = vnew > 0.0f ? __fdividef(vref, vnew) : 1.0f;
    const float ao0 = am0 * vr, ao1 = am1 * vr;
    vref = vnew;
    float ps0 = 0.0f, ps1 = 0.0f;
#pragma unroll
    for (int j = 0; j < 2 * kTileBlocks; ++j) {
      s[j][0] = ex2(s[j][0] - mu0); s[j][1] = ex2(s[j][1] - mu0);
      s[j][2] = ex2(s[j][2] - mu1); s[j][3] = ex2(s[j][3] - mu1);
      ps0 += s[j][0] + s[j][1];
      ps1 += s[j][2] + s[j][3];
    }
    l0 = l0 * am0 + ps0;
    l1 = l1 * am1 + ps1;
#pragma unroll
    for (int t = 0; t < kNTiles; ++t) {
      o[t][0] *= ao0; o[t][1] *= ao0;
      o[t][2] *= ao1; o[t][3] *= ao1;
    }

    // ---- O += P V ----------------------------------------------------------------------------------
#pragma unroll
    for (int jb = 0; jb < kTileBlocks; ++jb) {
      const float pv = vnew > 0.0f ? __fdividef(ts[2 * jb + 1], vnew) : 0.0f;
      const uint32_t pa0 = pack_f16x2(s[2 * jb][0] * pv, s[2 * jb][1] * pv);
      const uint32_t pa1 = pack_f16x2(s[2 * jb][2] * pv, s[2 * jb][3] * pv);
      const uint32_t pa2 = pack_f16x2(s[2 * jb + 1][0] * pv, s[2 * jb + 1][1] * pv);
      const uint32_t pa3 = pack_f16x2(s[2 * jb + 1][2] * pv, s[2 * jb + 1][3] * pv);
      const uint8_t* vp = cv + jb * C::kConvBlock + (D / 32) * 1024 + lane * 16;
#pragma unroll
      for (int qd = 0; qd < D / 32; ++qd) {
        const uint4 a = lds128(vp + qd * 1024);
        const uint4 c = lds128(vp + qd * 1024 + 512);
        mma16816<true>(o[4 * qd], pa0, pa1, pa2, pa3, a.x, a.y);
        mma16816<true>(o[4 * qd + 1], pa0, pa1, pa2, pa3, a.z, a.w);
        mma16816<true>(o[4 * qd + 2], pa0, pa1, pa2, pa3, c.x, c.y);
        mma16816<true>(o[4 * qd + 3], pa0, pa1, pa2, pa3, c.z, c.w);
      }
    }
  }

  if (failed) {
    if (tid == 0) atomicCAS(p.status, 0, COOPT_ERR_TIMEOUT);
    // copies still in flight get a bounded time to land before the shared memory is released
    for (int t = 0; t < issued; ++t) mbar_wait_bounded(&bars[t % kRawStages], (t / kRawStages) & 1u);
    return;
  }

  // ---- normalise and store -------------------------------------------------------------------------
  l0 = quad_sum(l0);
  l1 = quad_sum(l1);
  const float f0 = l0 > 0.0f ? vref / l0 : 0.0f, f1 = l1 > 0.0f ? vref / l1 : 0.0f;
  if (live0) {
    __nv_bfloat16* op = p.out + grow0 * D + 2 * quad;
#pragma unroll
    for (int t = 0; t < kNTiles; ++t)
      *reinterpret_cast<uint32_t*>(op + 8 * t) = pack_bf16x2(o[t][0] * f0, o[t][1] * f0);
  }
  if (live1) {
    __nv_bfloat16* op = p.out + grow1 * D + 2 * quad;
#pragma unroll
    for (int t = 0; t < kNTiles; ++t)
      *reinterpret_cast<uint32_t*>(op + 8 * t) = pack_bf16x2(o[t][2] * f1, o[t][3] * f1);
  }
}

template <int D>
int launch_prefill_one(const PrefillParams& p, dim3 grid, cudaStream_t stream) {
  using C = PfCfg<D>;
  if (!configure_kernel_smem(reinterpret_cast<const void*>(&paged_prefill_kernel<D>), C::kSmemBytes)) return COOPT_ERR_CUDA;
  paged_prefill_kernel<D><<<grid, kPfThreads, C::kSmemBytes, stream>>>(p);
  return cudaGetLastError() == cudaSuccess ? COOPT_OK : COOPT_ERR_CUDA;
}

}  // namespace

int launch_paged_prefill_umma(const coopt_cache* c, const void* q, void* out, const int32_t* cu_q_lens, const int32_t* block_table,
                              int32_t max_blocks_per_seq, const int32_t* context_lens, int32_t batch, int32_t num_q_heads,
                              int32_t total_q, int32_t causal, float sm_scale, void* workspace, cudaStream_t stream);

int launch_paged_prefill(const coopt_cache* c, const void* q, void* out, const int32_t* cu_q_lens,
                         const int32_t* block_table, int32_t max_blocks_per_seq, const int32_t* context_lens,
                         int32_t batch, int32_t num_q_heads, int32_t total_q, int32_t causal, float sm_scale,
                         void* workspace, cudaStream_t stream) {
  if (!is_fp8(c->dtype)) return COOPT_ERR_UNSUPPORTED;
  if (c->dtype == COOPT_KV_FP8_E5M2 && c->head_dim != 128) return COOPT_ERR_UNSUPPORTED;   // the E5M2 ablation: tcgen05 kernel only
  if (num_q_heads / c->num_kv_heads > kPfRows) return COOPT_ERR_UNSUPPORTED;   // a tile holds at least one query token of every head of the group
  // head_dim 128: the tcgen05 kernel; head_dim 64: the mma.sync kernel of this file
  if (c->head_dim == 128)
    return launch_paged_prefill_umma(c, q, out, cu_q_lens, block_table, max_blocks_per_seq, context_lens, batch, num_q_heads,
                                     total_q, causal, sm_scale, workspace, stream);
  PrefillParams p;
  p.cache = static_cast<const uint8_t*>(c->data);
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.out = static_cast<__nv_bfloat16*>(out);
  p.cu_q_lens = cu_q_lens;
  p.block_table = block_table;
  p.context_lens = context_lens;
  p.max_blocks_per_seq = max_blocks_per_seq;
  p.batch = batch;
  p.num_q_heads = num_q_heads;
  p.num_kv_heads = c->num_kv_heads;
  p.group = num_q_heads / c->num_kv_heads;
  p.num_blocks = c->num_blocks;
  p.tile_queries = kPfRows / p.group;
  p.causal = causal;
  p.sm_scale_log2 = sm_scale * kLog2e;
  p.status = static_cast<int*>(workspace);
  // every sequence adds at most one partly filled tile
  const long long tiles = static_cast<long long>(total_q) / p.tile_queries + batch;
  if (tiles > 0x7fffffffll) return COOPT_ERR_UNSUPPORTED;
  const dim3 grid(static_cast<unsigned>(tiles), static_cast<unsigned>(c->num_kv_heads));
  return c->head_dim == 128 ? launch_prefill_one<128>(p, grid, stream) : launch_prefill_one<64>(p, grid, stream);
}

}  // namespace coopt
