// Paged GQA decode over the FP8 cache on the 5th-generation tensor cores: Algorithm 1 phase 2
// (Eq. 6 dequantisation on load), Algorithm 2 (Eq. 7-8: the G query heads of a group consume one
// K/V stream), Algorithm 3 (Eq. 9 valid blocks only, Eq. 10 max-subtracted softmax) and the
// Opt-Pa chunk-and-merge reduction.
//
// The E4M3 codes of the cache are never widened by the SM's arithmetic pipes: they travel
// HBM -> shared memory (bulk async copies) -> tcgen05.mma kind::f8f6f4, whose products of two E4M3
// values are exact and whose accumulators are fp32 in tensor memory.  Both contractions are
// written "tokens first" so that the 128 rows of the instruction carry real work:
//     S^T [128 tokens x 16]   = Ktile [128 tokens x D] . Qg^T   (Qg: 16 rows = G heads x 2 terms)
//     O^T [D dims     x NP]  += Vt    [D x 128 tokens] . Pg^T   (Pg: NP rows = G heads x 3 terms)
// A bf16 query element (8 significant bits) is the exact sum of its nearest E4M3 value and the
// E4M3 value of the remainder; a probability is carried as three E4M3 terms (12 bits).  The K scale
// of a block multiplies the logits of its 16 tokens, the V scale is folded into the probabilities.
//
// One CTA per SM walks its slice of the flat (sequence, kv head, block) list in tiles of eight
// cache blocks.  Warp roles: warp 4 issues the copies of a tile (header, K part, V part of every
// granule) into a ring of stages; one lane of warp 5 issues the matrix instructions; warps 0-3 own
// the 128 tensor-memory lanes: thread t reads the logits of token t, takes part in the per-head
// maximum (warp shuffles, then one shared-memory step across the four warps), writes the
// probability terms of its token as one byte per row of Pg, rescales the running output when a
// maximum or the reference V scale grew, and at the end of a segment normalises dim t of the output.
// Every wait is bounded; a wait that runs out is reported in the workspace status word and all
// roles leave through the common exit, which frees the tensor memory.
#include "coopt_plan.cuh"

namespace coopt {

namespace {

constexpr int kUmmaThreads = 192;
constexpr int kSmThreads = 128;                       // warps 0-3
constexpr int kProducerWarp = 4, kMmaWarp = 5;
constexpr int kTileBlocks = 8;
constexpr int kTileTokens = kTileBlocks * kBlockSize;  // 128
constexpr int kTmemCols = 64;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kLog2eU = 1.4426950408889634f;

template <int D, int NP>
struct UCfg {
  static constexpr int kGran = granule_bytes(D, true);
  static constexpr int kPart = kBlockSize * D;                 // K (or V) codes of one granule
  static constexpr int kGMax = NP == 16 ? 5 : 8;               // head slots per probability term
  static constexpr int kStages = D == 128 ? 6 : 8;
  static constexpr int kKArea = kTileBlocks * kPart;
  static constexpr int kVArea = kTileBlocks * kPart + (D == 64 ? kPart : 0);   // D = 64: rows 64..127 of the 128-row operand read on
  static constexpr int kHdrArea = kTileBlocks * kFp8Header;
  static constexpr int kStageBytes = kKArea + kVArea + kHdrArea;
  static constexpr int kQBytes = 2 * 8 * D;                    // 16 rows x D codes
  static constexpr int kPBytes = NP * kTileTokens;             // NP rows x 128 codes
  // shared memory carve-up (bytes)
  static constexpr int kRingOff = 0;
  static constexpr int kQOff = kRingOff + kStages * kStageBytes;
  static constexpr int kPOff = kQOff + 2 * kQBytes;
  static constexpr int kIdsOff = kPOff + 2 * kPBytes;
  static constexpr int kPreBlkOff = kIdsOff + kCap * 4;
  static constexpr int kPreUnitOff = kPreBlkOff + (kMaxBatch + 4) * 4;
  static constexpr int kSegOff = kPreUnitOff + (kMaxBatch + 4) * 4;
  static constexpr int kRedOff = kSegOff + kMaxSeg * static_cast<int>(sizeof(Segment));   // float [2][4][8] + [4][8] + [4][8]
  static constexpr int kBarOff = kRedOff + (2 * 4 * 8 + 4 * 8 + 4 * 8) * 4;
  static constexpr int kNumBars = 2 * kStages + 2 + 2 + 2 + 2 + 1;
  static constexpr int kMiscOff = kBarOff + kNumBars * 8;
  static constexpr int kSmemBytes = kMiscOff + 64;
  static_assert(kSmemBytes <= 232448, "shared memory of one CTA");
};

// ---- tcgen05 wrappers ----------------------------------------------------------------------------
// Shared-memory operand descriptor, K-major, no swizzle: element (row r, byte k) of the operand sits
// at (r / 8) * sbo + (k / 16) * lbo + (r % 8) * 16 + k % 16 from the start address.
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
  return static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4) | (static_cast<uint64_t>(lbo >> 4) << 16) |
         (static_cast<uint64_t>(sbo >> 4) << 32) | (1ull << 46);
}
// Instruction descriptor: E4M3 x E4M3 -> fp32, both operands K-major, M = 128, N = n.
__device__ __forceinline__ constexpr uint32_t umma_idesc(int n) {
  return (1u << 4) | (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(128 >> 4) << 24);
}
__device__ __forceinline__ void umma_f8(uint32_t d_tmem, uint64_t a, uint64_t b, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n}"
               ::"r"(d_tmem), "l"(a), "l"(b), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
                 "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
               : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const float (&v)[16]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
               ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
                 "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])),
                 "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])),
                 "r"(__float_as_uint(v[11])), "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])),
                 "r"(__float_as_uint(v[15]))
               : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Barrier 1 of the 128 softmax threads, carrying an OR reduction of a per-thread flag.
__device__ __forceinline__ bool sm_barrier_or(bool flag) {
  uint32_t r;
  asm volatile("{\n .reg .pred p, q;\n setp.ne.b32 p, %1, 0;\n barrier.cta.red.or.pred q, 1, 128, p;\n selp.u32 %0, 1, 0, q;\n}"
               : "=r"(r) : "r"(static_cast<uint32_t>(flag)) : "memory");
  return r != 0;
}
// Bounded wait that also gives up when another role has already given up.
__device__ __forceinline__ bool wait_bar(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_timer_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag != 0) return false;
    if (global_timer_ns() - t0 > kWaitLimitNs) { *abort_flag = 1; return false; }
  }
}

__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
  return x;
}
__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}
// Two fp32 values -> two E4M3 codes (first argument in bits 0..7), round to nearest even, saturating.
__device__ __forceinline__ uint32_t f32x2_to_e4m3x2(float lo, float hi) {
  uint16_t d;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(d) : "f"(hi), "f"(lo));
  return d;
}
// codes = e4m3(lo), e4m3(hi); lo and hi are replaced by what the codes leave over (exact in fp32).
__device__ __forceinline__ uint32_t e4m3_term(float& lo, float& hi) {
  const uint32_t codes = f32x2_to_e4m3x2(lo, hi);
  const uint32_t back = e4m3x2_to_f16x2_lo(codes);
  lo -= __half2float(__ushort_as_half(static_cast<unsigned short>(back & 0xFFFFu)));
  hi -= __half2float(__ushort_as_half(static_cast<unsigned short>(back >> 16)));
  return codes;
}

template <int D, int NP>
__global__ void __launch_bounds__(kUmmaThreads, 1) paged_decode_umma_kernel(const DecodeParams p) {
  using C = UCfg<D, NP>;
  constexpr int kGMax = C::kGMax;
  constexpr int kKSteps = D / 32;                 // 32 codes per instruction along the contraction
  constexpr uint32_t kSboRows = 8 * D;            // 8 rows of D codes: stride between row groups of K, Q
  extern __shared__ __align__(128) uint8_t smem[];
  uint8_t* ring = smem + C::kRingOff;
  uint8_t* qbuf = smem + C::kQOff;
  uint8_t* pbuf = smem + C::kPOff;
  PlanSmem plan;
  plan.ids = reinterpret_cast<int*>(smem + C::kIdsOff);
  plan.pre_blk = reinterpret_cast<int*>(smem + C::kPreBlkOff);
  plan.pre_unit = reinterpret_cast<int*>(smem + C::kPreUnitOff);
  plan.segs = reinterpret_cast<Segment*>(smem + C::kSegOff);
  plan.misc = reinterpret_cast<int*>(smem + C::kMiscOff);          // [0..2] planner, [3] last-arriver flag
  float* red_max = reinterpret_cast<float*>(smem + C::kRedOff);    // [2][4][8]
  float* red_sum = red_max + 2 * 4 * 8;                            // [4][8]
  float* red_q = red_sum + 4 * 8;                                  // [4][8]
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::kBarOff);
  uint64_t* bar_full = bars;                        // [kStages] copies of a tile landed
  uint64_t* bar_empty = bar_full + C::kStages;      // [kStages] the P V instructions of the tile in this stage are done
  uint64_t* bar_sfull = bar_empty + C::kStages;     // [2] logits of a tile are in tensor memory
  uint64_t* bar_sfree = bar_sfull + 2;              // [2] the four softmax warps have read them
  uint64_t* bar_pfull = bar_sfree + 2;              // [2] probabilities of a tile are in shared memory, O rescaled
  uint64_t* bar_qfull = bar_pfull + 2;              // [2] query operand of a segment is in shared memory
  volatile int* abort_flag = plan.misc + 4;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(plan.misc + 5);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int B = p.batch, Hkv = p.num_kv_heads, G = p.group, Hq = p.num_q_heads;
  const bool chunk_mode = p.chunk_blocks > 0;

  // ---- set-up ---------------------------------------------------------------------------------------
  // operand areas start at zero: rows of Qg / Pg that no head uses and ring slots a short tile leaves
  // untouched must hold finite codes
  for (int i = tid; i < C::kIdsOff / 16; i += kUmmaThreads) reinterpret_cast<uint4*>(smem)[i] = make_uint4(0u, 0u, 0u, 0u);
  if (tid == 0) {
    for (int i = 0; i < C::kStages; ++i) { mbar_init(&bar_full[i], 1); mbar_init(&bar_empty[i], 1); }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bar_sfull[i], 1);
      mbar_init(&bar_sfree[i], 4);
      mbar_init(&bar_pfull[i], kSmThreads);
      mbar_init(&bar_qfull[i], kSmThreads);
    }
    mbar_fence_init();
    *abort_flag = 0;
  }
  if (warp == kMmaWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  plan_prefix(p, plan, tid, kUmmaThreads);
  // sequences with an empty context: all-zero output rows
  for (int b = blockIdx.x; b < B; b += gridDim.x) {
    if (plan.pre_blk[b + 1] == plan.pre_blk[b])
      for (int i = tid; i < Hq * D; i += kUmmaThreads) p.out[static_cast<size_t>(b) * Hq * D + i] = __float2bfloat16(0.0f);
  }
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tmem_s[2] = {tmem, tmem + 16};
  const uint32_t tmem_o = tmem + 32;
  const uint32_t lane_base = static_cast<uint32_t>(warp & 3) * 32u << 16;

  PlanSlice sl;
  const bool active = plan_slice(p, plan, sl);

  // counters that persist across rounds (every role advances them identically)
  uint32_t tile_no = 0;     // tiles processed so far: ring stage and S / P buffer parity
  uint32_t seg_no = 0;      // segments processed so far: Q buffer parity
  // softmax state of the next segment's query scales (softmax threads)
  float qs_cur[kGMax], qs_next[kGMax];
#pragma unroll
  for (int h = 0; h < kGMax; ++h) { qs_cur[h] = 0.0f; qs_next[h] = 0.0f; }
  // producer: parity bookkeeping for the drain on the failure path
  uint32_t issued_tiles = 0;

  long long x = active ? sl.lo : 0;
  const long long x_end = active ? sl.hi : 0;
  while (x < x_end) {
    if (tid == 0) plan_round(p, plan, sl, x);
    __syncthreads();
    const int nseg = plan.misc[0];
    const long long x_next = (static_cast<long long>(plan.misc[2]) << 32) | static_cast<unsigned int>(plan.misc[1]);
    plan_stage_ids(p, plan, nseg, tid, kUmmaThreads);
    __syncthreads();

    if (warp == kProducerWarp) {
      // ================= copies: header, K part and V part of every granule of a tile =================
      bool ok = true;
      for (int si = 0; si < nseg && ok; ++si) {
        const Segment sg = plan.segs[si];
        for (int k0 = 0; k0 < sg.n && ok; k0 += kTileBlocks) {
          const int nb = min(kTileBlocks, sg.n - k0);
          const uint32_t stage = issued_tiles % C::kStages, use = issued_tiles / C::kStages;
          if (use > 0) ok = wait_bar(&bar_empty[stage], (use - 1) & 1u, abort_flag);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          uint8_t* st = ring + stage * C::kStageBytes;
          if (lane == 0) mbar_expect_tx(&bar_full[stage], nb * C::kGran);
          __syncwarp();
          if (lane < 3 * nb) {
            const int i = lane / 3, part = lane - 3 * i;
            const int id = plan.ids[sg.list_off + k0 + i];
            const uint8_t* src = p.cache + (static_cast<size_t>(id) * Hkv + sg.g) * C::kGran;
            if (part == 0) bulk_copy_g2s(st + C::kKArea + C::kVArea + i * kFp8Header, src, kFp8Header, &bar_full[stage]);
            else if (part == 1) bulk_copy_g2s(st + i * C::kPart, src + kFp8Header, C::kPart, &bar_full[stage]);
            else bulk_copy_g2s(st + C::kKArea + i * C::kPart, src + kFp8Header + C::kPart, C::kPart, &bar_full[stage]);
          }
          ++issued_tiles;
        }
      }
      if (!ok && lane == 0) atomicCAS(p.status, 0, COOPT_ERR_TIMEOUT);
    } else if (warp == kMmaWarp) {
      // ================= matrix instructions (one lane) ====================================================
      if (lane == 0) {
        bool ok = true;
        // two cursors over the round's tiles: the logits run one tile ahead of P V
        int a_si = 0, a_k0 = 0;
        uint32_t a_tile = tile_no, a_seg = seg_no;
        auto a_normalise = [&]() { while (a_si < nseg && a_k0 >= plan.segs[a_si].n) { ++a_si; a_k0 = 0; ++a_seg; } };
        auto issue_s = [&]() {
          const uint32_t stage = a_tile % C::kStages, buf = a_tile & 1u, use = a_tile >> 1;
          ok = ok && wait_bar(&bar_full[stage], (a_tile / C::kStages) & 1u, abort_flag);
          if (ok && use > 0) ok = wait_bar(&bar_sfree[buf], (use - 1) & 1u, abort_flag);
          if (ok && a_k0 == 0) ok = wait_bar(&bar_qfull[a_seg & 1u], (a_seg >> 1) & 1u, abort_flag);
          if (!ok) return;
          tc_fence_after();
          const uint32_t ka = smem_u32(ring + stage * C::kStageBytes);
          const uint32_t qa = smem_u32(qbuf + (a_seg & 1u) * C::kQBytes);
#pragma unroll
          for (int ks = 0; ks < kKSteps; ++ks)
            umma_f8(tmem_s[buf], umma_desc(ka + ks * 256, 128, kSboRows), umma_desc(qa + ks * 256, 128, kSboRows), umma_idesc(16), ks > 0);
          umma_commit(&bar_sfull[buf]);
          ++a_tile;
          a_k0 += kTileBlocks;
        };
        a_normalise();
        if (a_si < nseg) { issue_s(); a_normalise(); }
        for (int si = 0; si < nseg && ok; ++si) {
          const int n = plan.segs[si].n;
          for (int k0 = 0; k0 < n && ok; k0 += kTileBlocks) {
            if (a_si < nseg) { issue_s(); a_normalise(); }
            if (!ok) break;
            const int nb = min(kTileBlocks, n - k0);
            const uint32_t stage = tile_no % C::kStages, buf = tile_no & 1u;
            ok = wait_bar(&bar_pfull[buf], (tile_no >> 1) & 1u, abort_flag);
            if (!ok) break;
            tc_fence_after();
            const uint32_t va = smem_u32(ring + stage * C::kStageBytes + C::kKArea);
            const uint32_t pa = smem_u32(pbuf + buf * C::kPBytes);
            const int nks = (nb + 1) >> 1;                  // 32 tokens (two granules) per instruction
            for (int ks = 0; ks < nks; ++ks)
              umma_f8(tmem_o, umma_desc(va + ks * 2 * C::kPart, C::kPart, 128), umma_desc(pa + ks * 256, 128, 1024), umma_idesc(NP),
                      (k0 > 0 || ks > 0) ? 1u : 0u);
            umma_commit(&bar_empty[stage]);     // the stage is free again and the running output holds this tile
            ++tile_no;
          }
          ++seg_no;
        }
        if (!ok) atomicCAS(p.status, 0, COOPT_ERR_TIMEOUT);
      }
    } else {
      // ================= softmax warps: thread t owns token t of a tile and dim t of the output ========
      const int t = tid;
      bool bad = false;     // warp-uniform: a wait of this warp ran out
      // query operand of a segment: E4M3 lead term in rows 0..7, remainder term in rows 8..15
      auto prepare_q = [&](const Segment& sg, uint32_t segc, float (&qs)[kGMax]) {
        uint8_t* qb = qbuf + (segc & 1u) * C::kQBytes;
        float xq[kGMax], am[kGMax];
#pragma unroll
        for (int h = 0; h < kGMax; ++h) {
          xq[h] = 0.0f;
          if (h < G && t < D) xq[h] = __bfloat162float(p.q[(static_cast<size_t>(sg.b) * Hq + sg.g * G + h) * D + t]);
          am[h] = warp_max(fabsf(xq[h]));
        }
        float* rm = red_q;
        if (lane == 0) {
#pragma unroll
          for (int h = 0; h < kGMax; ++h) rm[warp * 8 + h] = am[h];
        }
        bad = sm_barrier_or(bad);
#pragma unroll
        for (int h = 0; h < kGMax; ++h) {
          const float amax = fmaxf(fmaxf(rm[h], rm[8 + h]), fmaxf(rm[16 + h], rm[24 + h]));
          // exact power-of-two scaling of the row into [128, 256), undone on the logits
          int k2 = 0;
          if (amax > 0.0f) k2 = max(-64, min(64, 134 - static_cast<int>((__float_as_uint(amax) >> 23) & 0xFF)));
          const float up = __uint_as_float(static_cast<uint32_t>(k2 + 127) << 23);
          qs[h] = p.sm_scale_log2 * __uint_as_float(static_cast<uint32_t>(127 - k2) << 23);
          xq[h] *= up;
        }
        if (t < D) {
          const uint32_t col = (t >> 4) * 128 + (t & 15);
#pragma unroll
          for (int h = 0; h < kGMax; h += 2) {
            float a = xq[h], b = h + 1 < kGMax ? xq[h + 1] : 0.0f;
            const uint32_t lead = e4m3_term(a, b);
            const uint32_t rest = f32x2_to_e4m3x2(a, b);
            if (h < G) { qb[col + h * 16] = static_cast<uint8_t>(lead & 0xFF); qb[kSboRows + col + h * 16] = static_cast<uint8_t>(rest & 0xFF); }
            if (h + 1 < G) { qb[col + (h + 1) * 16] = static_cast<uint8_t>(lead >> 8); qb[kSboRows + col + (h + 1) * 16] = static_cast<uint8_t>(rest >> 8); }
          }
        }
        bad = sm_barrier_or(bad);      // every thread has read the exchange buffer before the next segment's query reuses it
        fence_proxy_async();
        mbar_arrive(&bar_qfull[segc & 1u]);
      };

      if (nseg > 0) prepare_q(plan.segs[0], seg_no, qs_next);
      for (int si = 0; si < nseg && !bad; ++si) {
        const Segment sg = plan.segs[si];
#pragma unroll
        for (int h = 0; h < kGMax; ++h) qs_cur[h] = qs_next[h];
        if (si + 1 < nseg) prepare_q(plan.segs[si + 1], seg_no + 1, qs_next);
        if (bad) break;

        float m_run[kGMax], l_run[kGMax];
#pragma unroll
        for (int h = 0; h < kGMax; ++h) { m_run[h] = -INFINITY; l_run[h] = 0.0f; }
        float vref = 0.0f;

        for (int k0 = 0; k0 < sg.n; k0 += kTileBlocks) {
          const int nb = min(kTileBlocks, sg.n - k0);
          const uint32_t stage = tile_no % C::kStages, buf = tile_no & 1u;
          uint8_t* st = ring + stage * C::kStageBytes;
          const float* hdr = reinterpret_cast<const float*>(st + C::kKArea + C::kVArea);
          const int tok0 = (sg.j0 + k0) * kBlockSize;
          const int ntok = min(nb * kBlockSize, sg.ctx_len - tok0);            // Eq. 9: tail of the context
          bool ok = !bad && wait_bar(&bar_sfull[buf], (tile_no >> 1) & 1u, abort_flag);
          ok = ok && wait_bar(&bar_full[stage], (tile_no / C::kStages) & 1u, abort_flag);
          ok = __all_sync(0xffffffffu, ok);
          bad = bad || !ok;
          float sc[kGMax];
          float sv = 0.0f;
          if (!bad) {
            tc_fence_after();
            float c[16];
            tmem_ld16(tmem_s[buf] + lane_base, c);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bar_sfree[buf]);
            const bool valid = t < ntok;
            const float sk = hdr[(t >> 4) * 8];
            sv = valid ? hdr[(t >> 4) * 8 + 1] : 0.0f;
#pragma unroll
            for (int h = 0; h < kGMax; ++h) {
              sc[h] = valid ? (c[h] + c[8 + h]) * (qs_cur[h] * sk) : -INFINITY;
              const float wm = warp_max(sc[h]);
              if (lane == 0) red_max[(buf * 4 + warp) * 8 + h] = wm;
            }
          }
          bad = sm_barrier_or(bad);
          if (bad) break;
          // reference V scale of the tile (uniform)
          float vmax = 0.0f;
#pragma unroll
          for (int i = 0; i < kTileBlocks; ++i)
            if (i * kBlockSize < ntok) vmax = fmaxf(vmax, hdr[i * 8 + 1]);
          const float vnew = fmaxf(vref, vmax);
          const float vr = vnew > 0.0f ? __fdividef(vref, vnew) : 1.0f;
          const float pvs = vnew > 0.0f ? __fdividef(sv, vnew) * 256.0f : 0.0f;   // probabilities are carried times 2^8
          vref = vnew;
          float a_o[kGMax], pw[kGMax];
          bool rescale = false;
          const float* rmx = red_max + buf * 32;
#pragma unroll
          for (int h = 0; h < kGMax; ++h) {
            const float m_tile = fmaxf(fmaxf(rmx[h], rmx[8 + h]), fmaxf(rmx[16 + h], rmx[24 + h]));
            const float m_new = fmaxf(m_run[h], m_tile);
            const float mu = m_new == -INFINITY ? 0.0f : m_new;
            const float a_m = ex2(m_run[h] - mu);
            const float pr = ex2(sc[h] - mu);
            l_run[h] = l_run[h] * a_m + pr;
            m_run[h] = m_new;
            a_o[h] = a_m * vr;
            pw[h] = pr * pvs;
            rescale = rescale || (h < G && a_o[h] != 1.0f);
          }
          // ---- running output: rescale what earlier tiles accumulated (thread t = dim t) ---------
          if (k0 > 0 && rescale) {
            const uint32_t prev = tile_no - 1;
            ok = !bad && wait_bar(&bar_empty[prev % C::kStages], (prev / C::kStages) & 1u, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            bad = bad || !ok;
            if (!bad) {
              tc_fence_after();
#pragma unroll
              for (int half = 0; half < NP / 16; ++half) {
                float o[16];
                tmem_ld16(tmem_o + lane_base + half * 16, o);
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                  const int col = half * 16 + j;
                  if (col < 3 * kGMax) o[j] *= a_o[col % kGMax];
                }
                tmem_st16(tmem_o + lane_base + half * 16, o);
              }
              tmem_st_wait();
              tc_fence_before();
            }
          }
          // ---- probabilities of token t: three E4M3 terms per head, one byte per row of Pg ----------
          if (!bad) {
            uint8_t* pb = pbuf + buf * C::kPBytes + (t >> 4) * 128 + (t & 15);
#pragma unroll
            for (int h = 0; h < kGMax; h += 2) {
              float a = pw[h], b = h + 1 < kGMax ? pw[h + 1] : 0.0f;
#pragma unroll
              for (int term = 0; term < 3; ++term) {
                const uint32_t codes = term < 2 ? e4m3_term(a, b) : f32x2_to_e4m3x2(a, b);
                const int r0 = term * kGMax + h, r1 = r0 + 1;
                if (h < G) pb[(r0 >> 3) * 1024 + (r0 & 7) * 16] = static_cast<uint8_t>(codes & 0xFF);
                if (h + 1 < G) pb[(r1 >> 3) * 1024 + (r1 & 7) * 16] = static_cast<uint8_t>(codes >> 8);
              }
            }
            // V codes of slots past the context inside the last block are cleared (row t = dim t of V^T)
            if ((ntok & 15) != 0 && t < D) {
              uint4* row = reinterpret_cast<uint4*>(st + C::kKArea + (ntok >> 4) * C::kPart + (t >> 3) * 128 + (t & 7) * 16);
              const int keep = ntok & 15;
              uint4 w = *row;
              uint32_t* ww = reinterpret_cast<uint32_t*>(&w);
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const int left = keep - 4 * j;
                ww[j] &= left >= 4 ? 0xFFFFFFFFu : (left <= 0 ? 0u : (1u << (8 * left)) - 1u);
              }
              *row = w;
            }
            fence_proxy_async();
            mbar_arrive(&bar_pfull[buf]);
          }
          ++tile_no;
        }
        // (a warp whose wait ran out in the last tile keeps company until the next barrier makes it known)

        // ---- end of segment: normalise dim t, write the output or the partial ---------------------
        const uint32_t last_tile = tile_no - 1;
        bool ok = !bad && wait_bar(&bar_empty[last_tile % C::kStages], (last_tile / C::kStages) & 1u, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        bad = bad || !ok;
        float acc[kGMax];
#pragma unroll
        for (int h = 0; h < kGMax; ++h) acc[h] = 0.0f;
        if (!bad) {
          tc_fence_after();
#pragma unroll
          for (int half = 0; half < NP / 16; ++half) {
            float o[16];
            tmem_ld16(tmem_o + lane_base + half * 16, o);
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const int col = half * 16 + j;
              if (col < 3 * kGMax) acc[col % kGMax] += o[j];
            }
          }
          tc_fence_before();
#pragma unroll
          for (int h = 0; h < kGMax; ++h) {
            const float ws = warp_sum(l_run[h]);
            if (lane == 0) red_sum[warp * 8 + h] = ws;
          }
        }
        bad = sm_barrier_or(bad);
        if (bad) break;
        const int h0 = sg.g * G;
        float* po = nullptr; float* pm = nullptr; float* pl = nullptr;
        size_t pstride = 1;
        if (sg.partial) {
          const size_t base = chunk_mode ? (static_cast<size_t>(sg.b) * Hq + h0) * p.max_chunks + sg.slot
                                         : static_cast<size_t>(sg.slot) * G;
          po = p.part_o + base * D; pm = p.part_m + base; pl = p.part_l + base;
          pstride = chunk_mode ? static_cast<size_t>(p.max_chunks) : 1;
        }
#pragma unroll
        for (int h = 0; h < kGMax; ++h) {
          if (h < G) {
            const float den = (red_sum[h] + red_sum[8 + h]) + (red_sum[16 + h] + red_sum[24 + h]);
            const float val = den > 0.0f ? acc[h] * (vref * (1.0f / 256.0f)) / den : 0.0f;
            if (!sg.partial) {
              if (t < D) p.out[(static_cast<size_t>(sg.b) * Hq + h0 + h) * D + t] = __float2bfloat16(val);
            } else {
              if (t < D) po[h * pstride * D + t] = val;
              if (t == 0) {
                pm[h * pstride] = chunk_mode ? m_run[h] * kLn2 : m_run[h];   // exported partials use natural-log units
                pl[h * pstride] = den;
              }
            }
          }
        }
        if (sg.partial) {
          __threadfence();
          bad = sm_barrier_or(bad);
          int* counter = p.counters + sg.b * Hkv + sg.g;
          if (t == 0) {
            const int old = atomicAdd(counter, 1);
            const int last = old == sg.expected - 1;
            if (last) *counter = 0;             // ready for the next call
            plan.misc[3] = last;
          }
          bad = sm_barrier_or(bad);
          if (plan.misc[3]) {
            // this CTA delivered the last piece: log-sum-exp merge of all pieces (split-K merge)
            __threadfence();
            int first_cta = 0;
            if (!chunk_mode) {
              const long long fs = static_cast<long long>(Hkv) * plan.pre_blk[sg.b] + static_cast<long long>(sg.g) * sg.seq_blocks;
              first_cta = plan_cta_of(sl, fs);
            }
            for (int idx = t; idx < G * D; idx += kSmThreads) {
              const int r = idx / D, d = idx % D;
              float M = -INFINITY;
              for (int c = 0; c < sg.expected; ++c) {
                const size_t at = chunk_mode ? (static_cast<size_t>(sg.b) * Hq + h0 + r) * p.max_chunks + c
                                             : static_cast<size_t>(2 * (first_cta + c) + (c == 0 ? 1 : 0)) * G + r;
                M = fmaxf(M, __ldcg(p.part_m + at));
              }
              float num = 0.0f, den = 0.0f;
              for (int c = 0; c < sg.expected; ++c) {
                const size_t at = chunk_mode ? (static_cast<size_t>(sg.b) * Hq + h0 + r) * p.max_chunks + c
                                             : static_cast<size_t>(2 * (first_cta + c) + (c == 0 ? 1 : 0)) * G + r;
                const float mc = __ldcg(p.part_m + at), lc = __ldcg(p.part_l + at);
                const float wgt = lc > 0.0f ? lc * (chunk_mode ? ex2((mc - M) * kLog2eU) : ex2(mc - M)) : 0.0f;
                num += wgt * __ldcg(p.part_o + at * D + d);
                den += wgt;
              }
              p.out[(static_cast<size_t>(sg.b) * Hq + h0 + r) * D + d] = __float2bfloat16(den > 0.0f ? num / den : 0.0f);
            }
          }
          bad = sm_barrier_or(bad);     // misc[3] and red_sum are reused by the next segment
        }
        ++seg_no;
      }
      if (bad && t == 0) atomicCAS(p.status, 0, COOPT_ERR_TIMEOUT);
    }

    __syncthreads();
    if (*abort_flag != 0) break;
    x = x_next;
    __syncthreads();
  }

  // ---- exit: copies still in flight get a bounded time to land, tensor memory is returned -----------
  if (*abort_flag != 0 && warp == kProducerWarp && lane == 0) {
    for (uint32_t s = 0; s < static_cast<uint32_t>(C::kStages) && s < issued_tiles; ++s) {
      const uint32_t last_use = (issued_tiles - 1 - s) / C::kStages;   // last use of stage (issued_tiles - 1 - s) % kStages
      mbar_wait_bounded(&bar_full[(issued_tiles - 1 - s) % C::kStages], last_use & 1u);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
}

template <int D, int NP>
int launch_umma_one(const DecodeParams& p, int grid, cudaStream_t stream) {
  using C = UCfg<D, NP>;
  static bool configured[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return COOPT_ERR_CUDA;
  if (dev < 64 && !configured[dev]) {
    if (cudaFuncSetAttribute(paged_decode_umma_kernel<D, NP>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes) != cudaSuccess)
      return COOPT_ERR_CUDA;
    configured[dev] = true;
  }
  paged_decode_umma_kernel<D, NP><<<grid, kUmmaThreads, C::kSmemBytes, stream>>>(p);
  return cudaGetLastError() == cudaSuccess ? COOPT_OK : COOPT_ERR_CUDA;
}

}  // namespace

// FP8 cache: group sizes 1..5 use 16 probability rows, 6..8 use 32.
int launch_paged_decode_umma(const DecodeParams& p, int head_dim, int grid, cudaStream_t stream) {
  if (p.group <= 5) return head_dim == 128 ? launch_umma_one<128, 16>(p, grid, stream) : launch_umma_one<64, 16>(p, grid, stream);
  return head_dim == 128 ? launch_umma_one<128, 32>(p, grid, stream) : launch_umma_one<64, 32>(p, grid, stream);
}

}  // namespace coopt
