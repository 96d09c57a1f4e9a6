// Paged GQA decode over the FP8 cache on the 5th-generation tensor cores: Algorithm 1 phase 2
// (Eq. 6 dequantisation on load), Algorithm 2 (Eq. 7-8: the G query heads of a group consume one
// K/V stream), Algorithm 3 (Eq. 9 valid blocks only, Eq. 10 max-subtracted softmax) and the
// Opt-Pa chunk-and-merge reduction.
//
// The E4M3 codes of the cache are never widened by the SM's arithmetic pipes: they travel
// HBM -> shared memory (bulk async copies) -> tcgen05.mma kind::f8f6f4, whose products of two E4M3
// values are exact and whose accumulators are fp32 in tensor memory.  Both contractions are
// written "tokens first" so that the 128 rows of the instruction carry real work:
//     S^T [128 tokens x 16]  = Ktile [128 tokens x D] . Qg^T   (Qg: 16 rows = G heads x 2 terms)
//     O^T [D dims     x NP]  = Vt    [D x 128 tokens] . Pg^T   (Pg: NP rows = G heads x 3 terms)
// A bf16 query element (8 significant bits) is the exact sum of its nearest E4M3 value and the
// E4M3 value of the remainder.  A probability is carried as three E4M3 terms, each holding what
// the earlier ones left over times 16 (12 bits in all, and tiny probabilities keep their bits).
// The K scale of a block multiplies the logits of its 16 tokens, the V scale is folded into the
// probabilities.
//
// One CTA per SM walks its slice of the flat (sequence, kv head, block) list in tiles of eight
// cache blocks (128 tokens).  Warp roles:
//   warp 8      issues the copies of a tile into a ring of stages, an mbarrier per stage counting the
//               bytes.  The cache is one 2-D tensor (row = granule) to the copy engine; one gather
//               request fetches the same columns of four granules (their K parts, their V parts, or
//               their headers), so a tile of eight granules costs six requests;
//   warps 9, 11 one lane each issues the matrix instructions of the logits (warp 9) and of the outputs
//               (warp 11) and commits them to mbarriers;
//   warps 0-3, 4-7   two softmax teams; even tiles go to team 0, odd tiles to team 1, so two tiles are
//               always in flight.  Thread t of a team reads the logits of token t from tensor memory,
//               takes part in the per-head maximum (one redux per head, then a shared-memory step
//               across the team's four warps), writes the probability terms of its token as one byte
//               per row of Pg, and owns dim t of the team's running output, kept in registers: the
//               P V product of each tile lands in a buffer of its own and is folded in one tile later,
//               so the tensor memory is never rescaled.  Each team keeps its own running maximum and
//               sum; at the end of a segment the two are merged like two split-KV pieces.
//   warp 10     the epilogue: merges the two teams' pieces of a segment, folds the consecutive segments of one
//               (sequence, kv head) that this CTA holds into a run (chunk mode: consecutive chunks, each also
//               exported as its own (m, l, o)), and writes a run that covers its sequence straight to the output.
// A run that does not cover its whole sequence leaves (m, l, o) in the workspace; the CTA that
// delivers the last piece merges all pieces by log-sum-exp and writes the bf16 output.
// What the CTA has to do comes from a plan (coopt_plan.cu) that one bulk copy brings into shared memory:
// its rounds of segments with the physical block ids already looked up.  A step that appends a token per
// sequence (Algorithm 1 phase 1 followed by phase 2 in one launch) lets team 1 write the new token's
// granule of every (sequence, kv head) whose last block lies in this CTA's slice -- no other CTA reads that
// block -- before the copy warp requests the tile that holds it.
// Every wait is bounded; a wait that runs out is reported in the workspace status word and all roles
// leave through the common exit, which frees the tensor memory.
#include <mutex>
#include <vector>

#include "coopt_plan.cuh"
#include "coopt_trace.cuh"
#include "coopt_umma.cuh"
#include "coopt_write.cuh"

namespace coopt {

namespace {

constexpr int kTeamThreads = 128;                     // four warps: one per 32 tensor-memory lanes
constexpr int kSmThreads = 2 * kTeamThreads;          // warps 0-7
constexpr int kProducerWarp = 8, kMmaWarp = 9, kEpilogueWarp = 10, kPvWarp = 11;
constexpr int kUmmaThreads = 384;
constexpr int kTileBlocks = 8;
constexpr int kTileTokens = kTileBlocks * kBlockSize;  // 128
constexpr float kLn2 = 0.6931471805599453f;

template <int D, int NP>
struct UCfg {
  static constexpr int kGran = granule_bytes(D, true);
  static constexpr int kPart = kBlockSize * D;                 // K (or V) codes of one granule
  static constexpr int kGatherRows = 4;                        // granules per gather request
  static constexpr int kGMax = NP == 16 ? 5 : 8;               // head slots per probability term
  static constexpr int kTmemCols = NP == 16 ? 128 : 256;       // 4 x 16 logits columns + 4 x NP output columns
  static constexpr int kStages = D == 128 ? (NP == 16 ? 6 : 5) : 8;
  static constexpr int kKArea = kTileBlocks * kPart;
  static constexpr int kVArea = kTileBlocks * kPart + (D == 64 ? kPart : 0);   // D = 64: rows 64..127 of the 128-row operand read on
  static constexpr int kHdrOff = kKArea + kVArea;               // the eight headers (scales) of the tile
  static constexpr int kStageBytes = kHdrOff + kTileBlocks * kFp8Header;
  static constexpr int kGroupBytes = kGatherRows * (2 * kPart + kFp8Header);   // what the three requests of four granules bring
  static constexpr int kQBytes = 2 * 8 * D;                    // 16 rows x D codes
  static constexpr int kQRawBytes = kGMax * D * 2;             // the bf16 query rows of one (sequence, kv head) as they sit in memory
  static constexpr int kPBytes = NP * kTileTokens;             // NP rows x 128 codes
  static constexpr int kXchFloats = kGMax * kTeamThreads;            // one team's output of a segment: [head][dim]
  static constexpr int kMlFloats = 4 * 8 + 8;                       // one team's sums (per warp) and maxima of a segment
  // shared memory carve-up (bytes)
  static constexpr int kRingOff = 0;
  static constexpr int kQOff = kRingOff + kStages * kStageBytes;
  static constexpr int kPOff = kQOff + 2 * kQBytes;
  static constexpr int kPlanOff = kPOff + 4 * kPBytes;             // one round of the plan: header, segments, block ids
  static constexpr int kQRawOff = kPlanOff + (kPlanRoundMax + 127) / 128 * 128;   // two segments' raw queries
  static constexpr int kXchOff = kQRawOff + 2 * kQRawBytes;
  static constexpr int kMlOff = kXchOff + 2 * kXchFloats * 4;       // [2 segment parities][2 teams][kMlFloats]
  static constexpr int kRedOff = kMlOff + 2 * 2 * kMlFloats * 4;
  // int red_max [2 teams][4 warps][12], uint red_q [4][8], float qscale [2][8]
  static constexpr int kRedBytes = (2 * 4 * 12 + 4 * 8 + 2 * 8) * 4;
  static constexpr int kBarOff = kRedOff + kRedBytes;
  static constexpr int kNumBars = 2 * kStages + 4 * 4 + 3 * 2 + 2 + 2;
  static constexpr int kWriteStage = 4 * kBlockSize * D;       // staging of team 1's four warps for the fused append
  static constexpr int kMiscOff = kBarOff + kNumBars * 8;
  static constexpr int kSmemBytes = kMiscOff + 128;            // flags, the tensor-memory address, the copy warp's first time stamp
  static_assert(kStageBytes % 128 == 0 && kKArea % 128 == 0 && kHdrOff % 128 == 0 && (kGatherRows * kPart) % 128 == 0 &&
                    (kGatherRows * kFp8Header) % 128 == 0, "tensor copies land on 128-byte boundaries");
  static_assert(kPart / 8 <= 256 && kGran % 16 == 0, "one box row is at most 256 eight-byte elements");
  static_assert(kSmemBytes <= 232448, "shared memory of one CTA");
  static_assert(kWriteStage <= kStageBytes && kPlanFirstChunk <= kPlanRoundMax && kPlanOff % 128 == 0, "staging areas");
};

// The CTA that delivered the last piece of a (sequence, kv head) merges all pieces by log-sum-exp (the
// split-KV merge) and writes the bf16 output rows.  One warp; lane l owns dims d0 = 4l .. 4l+3 of every
// head.  Two pieces at a time: all their (m, l, o) are loaded before any is used, so a batch costs one
// trip to L2; the running (M, num, den) carries over from batch to batch.  The first piece of a
// (sequence, kv head) sits in the odd slot of its CTA, the others in the even slot.
template <int D, int kGMax>
__device__ __forceinline__ void merge_run_pieces(const float* run_o, const float* run_m, const float* run_l, __nv_bfloat16* out_rows,
                                              int first_cta, int pieces, int G, int d0) {
  auto piece = [&](int c, int r) -> size_t { return (static_cast<size_t>(2 * (first_cta + c)) + (c == 0 ? 1 : 0)) * G + r; };
  float M[kGMax], den[kGMax];
  float4 nm[kGMax];
#pragma unroll
  for (int r = 0; r < kGMax; ++r) { M[r] = -INFINITY; den[r] = 0.0f; nm[r] = make_float4(0.0f, 0.0f, 0.0f, 0.0f); }
  for (int c0 = 0; c0 < pieces; c0 += 2) {
    float mc[2][kGMax], lc[2][kGMax];
    float4 oc[2][kGMax];
#pragma unroll
    for (int k = 0; k < 2; ++k)
#pragma unroll
      for (int r = 0; r < kGMax; ++r) {
        const bool on = r < G && c0 + k < pieces;
        const size_t at = on ? piece(c0 + k, r) : 0;
        mc[k][r] = on ? __ldcg(run_m + at) : 0.0f;
        lc[k][r] = on ? __ldcg(run_l + at) : 0.0f;
        oc[k][r] = on ? __ldcg(reinterpret_cast<const float4*>(run_o + at * D + d0)) : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
      }
#pragma unroll
    for (int k = 0; k < 2; ++k)
#pragma unroll
      for (int r = 0; r < kGMax; ++r) {
        if (lc[k][r] > 0.0f) {
          const float Mn = fmaxf(M[r], mc[k][r]);
          const float keep = ex2(M[r] - Mn), wgt = lc[k][r] * ex2(mc[k][r] - Mn);
          nm[r].x = nm[r].x * keep + wgt * oc[k][r].x;
          nm[r].y = nm[r].y * keep + wgt * oc[k][r].y;
          nm[r].z = nm[r].z * keep + wgt * oc[k][r].z;
          nm[r].w = nm[r].w * keep + wgt * oc[k][r].w;
          den[r] = den[r] * keep + wgt;
          M[r] = Mn;
        }
      }
  }
#pragma unroll
  for (int r = 0; r < kGMax; ++r) {
    if (r < G) {
      const float inv = den[r] > 0.0f ? 1.0f / den[r] : 0.0f;
      *reinterpret_cast<uint2*>(out_rows + static_cast<size_t>(r) * D + d0) =
          make_uint2(pack_bf16x2(nm[r].x * inv, nm[r].y * inv), pack_bf16x2(nm[r].z * inv, nm[r].w * inv));
    }
  }
}

template <int D, int NP>
__global__ void __launch_bounds__(kUmmaThreads, 1) paged_decode_umma_kernel(const DecodeParams p, const __grid_constant__ CUtensorMap map_part,
                                                                            const __grid_constant__ CUtensorMap map_hdr) {
  using C = UCfg<D, NP>;
  constexpr int kGMax = C::kGMax;
  constexpr int kKSteps = D / 32;                 // 32 codes per instruction along the contraction
  constexpr uint32_t kSboRows = 8 * D;            // 8 rows of D codes: stride between row groups of K, Q
  extern __shared__ __align__(128) uint8_t smem[];
  uint8_t* ring = smem + C::kRingOff;
  uint8_t* qbuf = smem + C::kQOff;
  uint8_t* pbuf = smem + C::kPOff;
  uint8_t* plan_smem = smem + C::kPlanOff;
  const PlanRound* round_hdr = reinterpret_cast<const PlanRound*>(plan_smem);
  PlanSmem plan;
  plan.segs = reinterpret_cast<Segment*>(plan_smem + 64);
  plan.ids = nullptr;                                               // behind the round's segments
  plan.pre_blk = plan.pre_unit = nullptr;
  plan.misc = reinterpret_cast<int*>(smem + C::kMiscOff);          // flags and the tensor-memory address
  plan.slice = nullptr;
  plan.bounds = nullptr;
  float* xch = reinterpret_cast<float*>(smem + C::kXchOff);         // [2 teams][kXchFloats]
  float* mlbuf = reinterpret_cast<float*>(smem + C::kMlOff);        // [2 segment parities][2 teams][kMlFloats]
  int* red_max = reinterpret_cast<int*>(smem + C::kRedOff);         // [2][4][12] per-warp maxima of a tile (ordered ints)
  uint32_t* red_q = reinterpret_cast<uint32_t*>(red_max + 2 * 4 * 12);   // [4][8]
  float* qscale = reinterpret_cast<float*>(red_q + 4 * 8);          // [2 segment parities][8] logit scale per head
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::kBarOff);
  uint64_t* bar_full = bars;                        // [kStages] copies of a tile landed
  uint64_t* bar_empty = bar_full + C::kStages;      // [kStages] the P V instructions of the tile in this stage are done
  uint64_t* bar_sfull = bar_empty + C::kStages;     // [4] logits of a tile are in tensor memory (buffer = tile & 3)
  uint64_t* bar_sfree = bar_sfull + 4;              // [4] the team's four warps have read them
  uint64_t* bar_pfull = bar_sfree + 4;              // [4] probabilities of a tile are in shared memory (buffer = tile & 3)
  uint64_t* bar_ofree = bar_pfull + 4;              // [4] the team has folded the output buffer into its registers
  uint64_t* bar_qfull = bar_ofree + 4;              // [2] query operand of a segment is in shared memory
  uint64_t* bar_efull = bar_qfull + 2;              // [2] both teams' pieces of a segment are in the exchange area
  uint64_t* bar_efree = bar_efull + 2;              // [2] the epilogue warp has read them
  uint64_t* bar_plan = bar_efree + 2;               // a piece of the plan has landed in shared memory
  uint64_t* bar_wdone = bar_plan + 1;               // team 1 has written the round's new tokens to the cache
  uint64_t* bar_qraw = bar_wdone + 1;               // [2] the raw query rows of a segment have landed (buffer = segment & 1)
  uint8_t* qraw = smem + C::kQRawOff;
  volatile int* abort_flag = plan.misc + 4;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(plan.misc + 5);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int B = p.batch, Hkv = p.num_kv_heads, G = p.group, Hq = p.num_q_heads;
  const bool chunk_mode = p.chunk_blocks > 0;

  // ---- set-up ---------------------------------------------------------------------------------------
  // two trips to memory start before anything else: the context lengths for the planner, and the copy
  // engine's view of the cache (fetched on first use otherwise, in front of the first tile)
  COOPT_TRACE_CYCLES(p.trace, kTrEntry, tid == 0);
#ifdef COOPT_TRACE
  if (tid == 0 && p.trace != nullptr && blockIdx.x < kTraceMaxCtas) trace_put(p.trace, kTrPrevExitNs, p.trace[blockIdx.x * kTraceSlots + kTrExitNs]);
#endif
  COOPT_TRACE_NS(p.trace, kTrEntryNs, tid == 0);
#ifdef COOPT_TRACE
  if (tid == 0) { unsigned int smid; asm volatile("mov.u32 %0, %%smid;" : "=r"(smid)); trace_put(p.trace, kTrSmId, smid + 1); }
#endif
#ifdef COOPT_TRACE
  const uint8_t* plan_region = p.plan + static_cast<size_t>((blockIdx.x + p.plan_rotate) % gridDim.x) * p.plan_cta_stride;
#else
  const uint8_t* plan_region = p.plan + static_cast<size_t>(blockIdx.x) * p.plan_cta_stride;
#endif
  if (tid == kProducerWarp * 32) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_part) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_hdr) : "memory");
  }
  // rows of Qg / Pg that no head uses must hold zero codes
  for (int i = tid; i < (C::kPlanOff - C::kQOff) / 16; i += kUmmaThreads)
    reinterpret_cast<uint4*>(smem + C::kQOff)[i] = make_uint4(0u, 0u, 0u, 0u);
  if (tid == 0) {
    for (int i = 0; i < C::kStages; ++i) { mbar_init(&bar_full[i], 1); mbar_init(&bar_empty[i], 1); }
    for (int i = 0; i < 4; ++i) {
      mbar_init(&bar_sfull[i], 1);
      mbar_init(&bar_sfree[i], 4);
      mbar_init(&bar_pfull[i], kTeamThreads);
      mbar_init(&bar_ofree[i], 4);
    }
    for (int i = 0; i < 2; ++i) { mbar_init(&bar_qfull[i], kTeamThreads); mbar_init(&bar_efull[i], kSmThreads); mbar_init(&bar_efree[i], 1); }
    mbar_init(bar_plan, 1);
    mbar_init(bar_wdone, 4);
    mbar_init(&bar_qraw[0], 1);
    mbar_init(&bar_qraw[1], 1);
    mbar_fence_init();
    *abort_flag = 0;
    // the first round of this CTA's plan: its size is not known yet, so a fixed first piece is fetched
    mbar_expect_tx(bar_plan, kPlanFirstChunk);
    bulk_copy_g2s(plan_smem, plan_region, kPlanFirstChunk, bar_plan);
  }
  if (warp == kMmaWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(C::kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  // Launched as a programmatic dependent of the kernel before it, this CTA may have started while that kernel
  // still runs.  Only the copy warp goes ahead (the plan and the cache blocks it requests were complete before
  // that kernel began); every other role waits here for it to finish, because the queries, the new tokens, the
  // output and the workspace may all be its results.  Without such a launch the wait returns at once.
  if (warp != kProducerWarp) asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  plan_check_single_query(p, tid, kUmmaThreads);
  COOPT_TRACE_CYCLES(p.trace, kTrSetupDone, tid == 0);
  const uint32_t tmem_o = tmem + 64;                           // logits buffer b at column 16 b, output buffer b at 64 + NP b
  const uint32_t lane_base = static_cast<uint32_t>(warp & 3) * 32u << 16;

  const bool has_new = p.k_new != nullptr;      // this launch also appends one token per sequence
  // counters that persist across rounds (every role advances its own copy identically)
  uint32_t tile_no = 0;     // tiles so far: ring stage, and team / buffer = tile_no & 1
  uint32_t seg_no = 0;      // segments so far: parity of the Q buffer and of the exchange area

  uint32_t round_no = 0, plan_phase = 0;
  size_t plan_at = 0;                            // where the current round starts in the CTA's plan region
  for (;;) {
    // ---- this round of the plan: what the first fetch did not bring is fetched now ---------------------
    bool plan_ok = wait_bar(bar_plan, plan_phase & 1u, abort_flag);
    ++plan_phase;
    const int round_bytes = plan_ok ? round_hdr->bytes : 0;
    if (plan_ok && round_bytes > kPlanFirstChunk) {
      if (tid == 0) {
        mbar_expect_tx(bar_plan, round_bytes - kPlanFirstChunk);
        bulk_copy_g2s(plan_smem + kPlanFirstChunk, plan_region + plan_at + kPlanFirstChunk, round_bytes - kPlanFirstChunk, bar_plan);
      }
      plan_ok = wait_bar(bar_plan, plan_phase & 1u, abort_flag);
      ++plan_phase;
    }
    // A wait that ran out has raised the abort flag: this thread skips the round's work (nseg = 0 below) but
    // keeps the CTA's barriers company, and everybody leaves behind the round's closing barrier.
    if (!plan_ok && lane == 0) atomicCAS(p.status, 0, COOPT_ERR_TIMEOUT);
    const bool plan_valid = plan_ok && round_hdr->key == p.plan_key && round_hdr->nseg <= kMaxSeg && round_bytes <= kPlanRoundMax &&
                            round_hdr->n_ids <= kCap;
    if (plan_ok && !plan_valid) {                                                // not a plan of this problem (the same verdict in every thread)
      if (tid == 0) atomicCAS(p.status, 0, COOPT_ERR_INVALID_ARG);
      break;
    }
    if (plan_ok && tid == 0 && round_hdr->status != 0) atomicCAS(p.status, 0, round_hdr->status);   // what the planner found
    const int nseg = plan_ok ? round_hdr->nseg : 0;
    if (warp == kEpilogueWarp && round_no == 0 && plan_ok) {
      // sequences with an empty context: all-zero output rows (this warp has nothing else to do yet, and no
      // other role waits for it here)
      for (int b = blockIdx.x; b < B; b += gridDim.x) {
        if ((p.plan_header->empty_bits[b >> 5] >> (b & 31)) & 1u) {
          uint4* row = reinterpret_cast<uint4*>(p.out + static_cast<size_t>(b) * Hq * D);
          for (int i = lane; i < Hq * D / 8; i += 32) row[i] = make_uint4(0u, 0u, 0u, 0u);
        }
      }
    }
    if (plan_ok && nseg <= 0) break;                                             // nothing (left) to do
    const bool last_round = !plan_ok || round_hdr->last != 0;
    plan.ids = reinterpret_cast<int*>(plan_smem + 64 + nseg * 64);
    const uint32_t round_tile0 = tile_no;             // every role's tile counter agrees at the start of a round
    uint8_t* write_stage = ring + ((round_tile0 + C::kStages - 1) % C::kStages) * C::kStageBytes;   // the stage the ring fills last
    COOPT_TRACE_CYCLES(p.trace, kTrIdsStaged, tid == 0 && round_no == 0);
    COOPT_TRACE_VALUE(p.trace, kTrNumSeg, tid == 0 && round_no == 0, nseg);

    if (warp == kProducerWarp) {
      // ================= copies: six gather requests per tile ==================================================
      // Lane 3 q + w (q = 0, 1; w = 0, 1, 2) fetches the K parts (w = 0), the V parts (w = 1) or the headers
      // (w = 2) of granules 4 q .. 4 q + 3 of the tile.  Rows past the tile's last granule repeat its first
      // one: their tokens are masked out of the softmax.  The rows of a tile are worked out before the lane
      // that watches the ring looks at the stage, so that the copy engine's queue is refilled with as little
      // of a gap as possible.
      bool ok = true;
      const int q4 = lane / 3, what = lane - 3 * q4;
      const int x = what * (C::kPart / 8);                    // first column, in 8-byte elements
      const uint32_t dst_off = what == 0 ? q4 * C::kGatherRows * C::kPart
                             : what == 1 ? C::kKArea + q4 * C::kGatherRows * C::kPart
                                         : C::kHdrOff + q4 * C::kGatherRows * kFp8Header;
      const CUtensorMap* map = what == 2 ? &map_hdr : &map_part;
      // A step that appends tokens: the tile that holds a sequence's last block, and the ring stage that
      // team 1 borrows as staging, are not requested before team 1 has written the round's new tokens.
      bool writes_pending = has_new && round_hdr->n_tail > 0;
      COOPT_TRACE_CYCLES(p.trace, kTrProducerPlan, lane == 0 && round_no == 0);

      for (int si = 0; si < nseg && ok; ++si) {
        const int n = plan.segs[si].n, g = plan.segs[si].g;
        const bool seg_tail = (plan.segs[si].run_flags & kSegTail) != 0;
        const int* seg_ids = plan.ids + plan.segs[si].list_off;
        for (int k0 = 0; k0 < n; k0 += kTileBlocks) {
          if (writes_pending && ((seg_tail && k0 + kTileBlocks >= n) || tile_no - round_tile0 == C::kStages - 1)) {
            if (lane == 0) ok = wait_bar(bar_wdone, round_no & 1u, abort_flag);
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            writes_pending = false;
          }
          const int nb = min(kTileBlocks, n - k0);
          const int ngroups = (nb + C::kGatherRows - 1) / C::kGatherRows;
          int rows[C::kGatherRows] = {0, 0, 0, 0};
          if (lane < 3 * ngroups) {
#pragma unroll
            for (int i = 0; i < C::kGatherRows; ++i) {
              const int j = q4 * C::kGatherRows + i;
              rows[i] = seg_ids[k0 + (j < nb ? j : 0)] * Hkv + g;
            }
          }
          const uint32_t stage = tile_no % C::kStages, use = tile_no / C::kStages;
          uint8_t* st = ring + stage * C::kStageBytes;
          if (lane == 0) {
            if (use > 0) ok = wait_bar(&bar_empty[stage], (use - 1) & 1u, abort_flag);
            if (ok) mbar_expect_tx(&bar_full[stage], ngroups * C::kGroupBytes);
          }
          ok = __shfl_sync(0xffffffffu, ok, 0);
          if (!ok) break;
          COOPT_TRACE_CYCLES(p.trace, kTrFirstCopyReady, lane == 0 && tile_no == 0);
          if (lane < 3 * ngroups) gather4_g2s(st + dst_off, map, x, rows[0], rows[1], rows[2], rows[3], &bar_full[stage]);
          COOPT_TRACE_CYCLES(p.trace, kTrFirstCopy, lane == 0 && tile_no == 0);
          COOPT_TRACE_CYCLES(p.trace, kTrLastCopy, lane == 0);
          COOPT_TRACE_CYCLES(p.trace, kTrCopyTileBase + static_cast<int>(tile_no), lane == 0 && tile_no < 32);
          ++tile_no;
        }
      }
      COOPT_TRACE_VALUE(p.trace, kTrNumTiles, lane == 0, tile_no);
      if (!ok && lane == 0) atomicCAS(p.status, 0, COOPT_ERR_TIMEOUT);
    } else if (warp == kMmaWarp) {
      // ================= logits: S^T = Ktile . Qg^T (one lane) ================================================
      // Runs ahead of the softmax teams by up to four tiles (four logits buffers).  A single thread issues
      // few instructions per cycle, so the two kinds of matrix instruction have a lane (and a warp
      // scheduler) each, and the operand descriptors of a tile are one addition away from constants.
      if (lane == 0) {
        bool ok = true;
        const uint64_t desc_k = umma_desc(smem_u32(ring), 128, kSboRows), desc_q = umma_desc(smem_u32(qbuf), 128, kSboRows);
        for (int si = 0; si < nseg && ok; ++si, ++seg_no) {
          const int n = plan.segs[si].n;
          ok = wait_bar(&bar_qfull[seg_no & 1u], (seg_no >> 1) & 1u, abort_flag);
          const uint64_t dq = desc_q + (((seg_no & 1u) * C::kQBytes) >> 4);
          for (int k0 = 0; k0 < n && ok; k0 += kTileBlocks, ++tile_no) {
            const uint32_t stage = tile_no % C::kStages, buf = tile_no & 3u, use = tile_no >> 2;
            ok = wait_bar(&bar_full[stage], (tile_no / C::kStages) & 1u, abort_flag);
            if (ok && use > 0) ok = wait_bar(&bar_sfree[buf], (use - 1) & 1u, abort_flag);
            if (!ok) break;
            COOPT_TRACE_CYCLES(p.trace, kTrFirstLanded, tile_no == 0);
            COOPT_TRACE_CYCLES(p.trace, kTrLastLanded, true);
            tc_fence_after();
            const uint64_t dk = desc_k + ((stage * C::kStageBytes) >> 4);
#pragma unroll
            for (int ks = 0; ks < kKSteps; ++ks) umma_f8(tmem + 16 * buf, dk + ks * 16, dq + ks * 16, umma_idesc(16, p.kv_e5m2), ks > 0);
            umma_commit(&bar_sfull[buf]);
            COOPT_TRACE_CYCLES(p.trace, kTrLogitsTileBase + static_cast<int>(tile_no), tile_no < 32);
          }
        }
        if (!ok) atomicCAS(p.status, 0, COOPT_ERR_TIMEOUT);
      }
    } else if (warp == kPvWarp) {
      // ================= outputs: O^T = V^T . Pg^T of a tile into its own buffer (one lane) ==================
      if (lane == 0) {
        bool ok = true;
        const uint64_t desc_v = umma_desc(smem_u32(ring + C::kKArea), C::kPart, 128), desc_p = umma_desc(smem_u32(pbuf), 128, 1024);
        for (int si = 0; si < nseg && ok; ++si) {
          const int n = plan.segs[si].n;
          for (int k0 = 0; k0 < n && ok; k0 += kTileBlocks, ++tile_no) {
            const uint32_t stage = tile_no % C::kStages, buf = tile_no & 3u, use = tile_no >> 2;
            ok = wait_bar(&bar_pfull[buf], use & 1u, abort_flag);
            if (ok && use > 0) ok = wait_bar(&bar_ofree[buf], (use - 1) & 1u, abort_flag);
            if (!ok) break;
            tc_fence_after();
            const uint64_t dv = desc_v + ((stage * C::kStageBytes) >> 4), dp = desc_p + ((buf * C::kPBytes) >> 4);
            const int nks = (min(kTileBlocks, n - k0) + 1) >> 1;      // 32 tokens (two granules) per instruction
            for (int ks = 0; ks < nks; ++ks)
              umma_f8(tmem_o + NP * buf, dv + ks * ((2 * C::kPart) >> 4), dp + ks * 16, umma_idesc(NP, p.kv_e5m2), ks > 0 ? 1u : 0u);
            umma_commit(&bar_empty[stage]);     // the stage is free again and the tile's product is in its output buffer
            COOPT_TRACE_CYCLES(p.trace, kTrLastPv, true);
            COOPT_TRACE_CYCLES(p.trace, kTrPvTileBase + static_cast<int>(tile_no), tile_no < 32);
          }
        }
        if (!ok) atomicCAS(p.status, 0, COOPT_ERR_TIMEOUT);
      }
    } else if (warp == kEpilogueWarp) {
      // ================= stores, piece counting and the split-KV merge: off the teams' critical path ========
      // Lane l owns dims 4l .. 4l+3 of every head.  A run (what this CTA holds of one (sequence, kv head):
      // one segment in decode mode, several consecutive chunks in chunk mode) is merged in registers; only
      // runs that do not cover their whole sequence go through the workspace and the piece counter.
      bool ok = true;
      const int d0 = lane * 4;
      float4 acc[kGMax];                    // the run so far: sum of weight * o, relative to acc_m
      float acc_m[kGMax], acc_l[kGMax];
#pragma unroll
      for (int h = 0; h < kGMax; ++h) { acc[h] = make_float4(0.0f, 0.0f, 0.0f, 0.0f); acc_m[h] = -INFINITY; acc_l[h] = 0.0f; }
      for (int si = 0; si < nseg; ++si, ++seg_no) {
        const Segment sg = plan.segs[si];
        const uint32_t par = seg_no & 1u;
        ok = wait_bar(&bar_efull[par], (seg_no >> 1) & 1u, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        COOPT_TRACE_CYCLES(p.trace, kTrLastHandOff, lane == 0);
        COOPT_TRACE_CYCLES(p.trace, kTrSegBase + static_cast<int>(seg_no), lane == 0 && seg_no < 20);
        const int h0 = sg.g * G;
        const size_t run_base = static_cast<size_t>(sg.run_slot) * G;
        // a run that an earlier round of this CTA began: its state was parked in the run's workspace slot
        if (si == 0 && !(sg.run_flags & kRunFirst)) {
#pragma unroll
          for (int h = 0; h < kGMax; ++h) {
            if (h < G) {
              if (d0 < D) acc[h] = *reinterpret_cast<const float4*>(p.run_o + (run_base + h) * D + d0);
              acc_m[h] = p.run_m[run_base + h];
              acc_l[h] = p.run_l[run_base + h];
            }
          }
        }
        // The two teams' running softmaxes are two pieces of the same segment.
        const float* ml = mlbuf + par * 2 * C::kMlFloats;
        float4 num[kGMax];
        float Mh[kGMax], denh[kGMax];
#pragma unroll
        for (int h = 0; h < kGMax; ++h) {
          num[h] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
          Mh[h] = -INFINITY;
          denh[h] = 0.0f;
          if (h < G) {
            const float* a0 = ml, *a1 = ml + C::kMlFloats;
            const float m0 = a0[32 + h], m1 = a1[32 + h];
            const float l0 = (a0[h] + a0[8 + h]) + (a0[16 + h] + a0[24 + h]), l1 = (a1[h] + a1[8 + h]) + (a1[16 + h] + a1[24 + h]);
            const float M = fmaxf(m0, m1);
            const float mu = M == -INFINITY ? 0.0f : M;
            const float w0 = ex2(m0 - mu) * (1.0f / 256.0f), w1 = ex2(m1 - mu) * (1.0f / 256.0f);   // outputs are carried times 2^8
            Mh[h] = M;
            denh[h] = (l0 * w0 + l1 * w1) * 256.0f;
            if (d0 < D) {
              const float4 v0 = *reinterpret_cast<const float4*>(xch + h * kTeamThreads + d0);
              const float4 v1 = *reinterpret_cast<const float4*>(xch + C::kXchFloats + h * kTeamThreads + d0);
              num[h] = make_float4(v0.x * w0 + v1.x * w1, v0.y * w0 + v1.y * w1, v0.z * w0 + v1.z * w1, v0.w * w0 + v1.w * w1);
            }
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&bar_efree[par]);      // the exchange area may take the next segment

        if (chunk_mode) {
          // Opt-Pa: the chunk's own (m, l, o) is exported, in natural-log units, o normalised
          const size_t base = (static_cast<size_t>(sg.b) * Hq + h0) * p.max_chunks + sg.slot;
#pragma unroll
          for (int h = 0; h < kGMax; ++h) {
            if (h < G) {
              const float inv = denh[h] > 0.0f ? 1.0f / denh[h] : 0.0f;
              const size_t at = base + static_cast<size_t>(h) * p.max_chunks;
              if (d0 < D) *reinterpret_cast<float4*>(p.part_o + at * D + d0) = make_float4(num[h].x * inv, num[h].y * inv, num[h].z * inv, num[h].w * inv);
              if (lane == 0) { p.part_m[at] = Mh[h] * kLn2; p.part_l[at] = denh[h]; }
            }
          }
        }
        // fold the segment into the run
#pragma unroll
        for (int h = 0; h < kGMax; ++h) {
          const float Mn = fmaxf(acc_m[h], Mh[h]);
          const float mu = Mn == -INFINITY ? 0.0f : Mn;
          const float ka = ex2(acc_m[h] - mu), kc = ex2(Mh[h] - mu);
          acc[h] = make_float4(acc[h].x * ka + num[h].x * kc, acc[h].y * ka + num[h].y * kc, acc[h].z * ka + num[h].z * kc, acc[h].w * ka + num[h].w * kc);
          acc_l[h] = acc_l[h] * ka + denh[h] * kc;
          acc_m[h] = Mn;
        }
        if (!(sg.run_flags & kRunLast)) {
          // the run goes on; if the round ends here, park it where its merged piece will go later (a run that
          // covers its whole sequence has no such slot: the CTA's second slot is free until a later run ends)
          if (si == nseg - 1) {
#pragma unroll
            for (int h = 0; h < kGMax; ++h) {
              if (h < G) {
                if (d0 < D) *reinterpret_cast<float4*>(p.run_o + (run_base + h) * D + d0) = acc[h];
                if (lane == 0) { p.run_m[run_base + h] = acc_m[h]; p.run_l[run_base + h] = acc_l[h]; }
              }
            }
            __syncwarp();
          }
          continue;
        }
        if (sg.run_flags & kRunWhole) {
          if (d0 < D) {
#pragma unroll
            for (int h = 0; h < kGMax; ++h) {
              if (h < G) {
                const float inv = acc_l[h] > 0.0f ? 1.0f / acc_l[h] : 0.0f;
                *reinterpret_cast<uint2*>(p.out + (static_cast<size_t>(sg.b) * Hq + h0 + h) * D + d0) =
                    make_uint2(pack_bf16x2(acc[h].x * inv, acc[h].y * inv), pack_bf16x2(acc[h].z * inv, acc[h].w * inv));
              }
            }
          }
#pragma unroll
          for (int h = 0; h < kGMax; ++h) { acc[h] = make_float4(0.0f, 0.0f, 0.0f, 0.0f); acc_m[h] = -INFINITY; acc_l[h] = 0.0f; }
          continue;
        }
        // the run is one piece of its (sequence, kv head): normalised o, maximum (base-2 units) and sum
#pragma unroll
        for (int h = 0; h < kGMax; ++h) {
          if (h < G) {
            const float inv = acc_l[h] > 0.0f ? 1.0f / acc_l[h] : 0.0f;
            if (d0 < D) *reinterpret_cast<float4*>(p.run_o + (run_base + h) * D + d0) = make_float4(acc[h].x * inv, acc[h].y * inv, acc[h].z * inv, acc[h].w * inv);
            if (lane == 0) { p.run_m[run_base + h] = acc_m[h]; p.run_l[run_base + h] = acc_l[h]; }
          }
        }
#pragma unroll
        for (int h = 0; h < kGMax; ++h) { acc[h] = make_float4(0.0f, 0.0f, 0.0f, 0.0f); acc_m[h] = -INFINITY; acc_l[h] = 0.0f; }
        __syncwarp();                         // every store of the piece has been issued
        COOPT_TRACE_CYCLES(p.trace, kTrPieceStored, lane == 0);
        int last = 0;
        if (lane == 0) {
          // release (this CTA's piece is visible before the count moves) and acquire (the other pieces
          // are visible before they are read) in one round trip
          int* counter = p.counters + sg.b * Hkv + sg.g;
          int old;
          asm volatile("atom.add.acq_rel.gpu.s32 %0, [%1], 1;" : "=r"(old) : "l"(counter) : "memory");
          last = old == sg.run_expected - 1;
          if (last) *counter = 0;             // ready for the next call
        }
        last = __shfl_sync(0xffffffffu, last, 0);
        COOPT_TRACE_CYCLES(p.trace, kTrCounted, lane == 0);
        if (last && d0 < D)
          merge_run_pieces<D, kGMax>(p.run_o, p.run_m, p.run_l, p.out + (static_cast<size_t>(sg.b) * Hq + h0) * D, sg.first_cta, sg.run_expected, G, d0);
      }
      COOPT_TRACE_CYCLES(p.trace, kTrEpilogueDone, lane == 0);
      if (!ok && lane == 0) atomicCAS(p.status, 0, COOPT_ERR_TIMEOUT);
    } else {
      // ================= softmax teams: thread t owns token t of its tiles and dim t of its output =====
      const int team = warp >> 2, wq = warp & 3;
      const int t = tid & (kTeamThreads - 1);
      const int team_bar = 1 + team;
      bool bad = false;     // warp-uniform until a barrier makes it uniform over the team
      bool team_bad = false;   // uniform over the team: set only behind such a barrier
      int* my_red_max = red_max + team * 48;

      // query operand of a segment (team 0): E4M3 lead term in rows 0..7, remainder term in rows 8..15.
      // The bf16 rows are brought into shared memory by a small bulk copy two segments ahead (fetch_q, one
      // thread), so that no thread of the team ever waits on a load from a memory system that the cache stream
      // keeps saturated; publish_q turns them into the operand behind the team's first tile of the segment before.
      auto fetch_q = [&](const Segment& sg, uint32_t segc) {
        const uint32_t bytes = static_cast<uint32_t>(G) * D * 2;
        fence_proxy_async();
        mbar_expect_tx(&bar_qraw[segc & 1u], bytes);
        bulk_copy_g2s(qraw + (segc & 1u) * C::kQRawBytes, p.q + (static_cast<size_t>(sg.b) * Hq + sg.g * G) * D, bytes, &bar_qraw[segc & 1u]);
      };
      float xq[kGMax];
      auto publish_q = [&](uint32_t segc, int si_next2) {
        uint8_t* qb = qbuf + (segc & 1u) * C::kQBytes;
        {
          bool ok = !bad && wait_bar(&bar_qraw[segc & 1u], (segc >> 1) & 1u, abort_flag);
          ok = __all_sync(0xffffffffu, ok);
          bad = bad || !ok;
          const __nv_bfloat16* raw = reinterpret_cast<const __nv_bfloat16*>(qraw + (segc & 1u) * C::kQRawBytes);
#pragma unroll
          for (int h = 0; h < kGMax; ++h) xq[h] = (!bad && h < G && t < D) ? __bfloat162float(raw[h * D + t]) : 0.0f;
        }
#pragma unroll
        for (int h = 0; h < kGMax; ++h) {
          const uint32_t am = __reduce_max_sync(0xffffffffu, __float_as_uint(fabsf(xq[h])));   // non-negative floats order like their bits
          if (lane == 0) red_q[wq * 8 + h] = am;
        }
        bad = barrier_or(team_bar, kTeamThreads, bad);
        uint32_t h2[(kGMax + 1) / 2];
#pragma unroll
        for (int h = 0; h < kGMax; h += 2) {
          float xs[2];
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const int hh = h + e < kGMax ? h + e : h;
            const uint32_t amax = max(max(red_q[hh], red_q[8 + hh]), max(red_q[16 + hh], red_q[24 + hh]));
            // exact power-of-two scaling of the row into [128, 256), undone on the logits
            int k2 = 0;
            if (amax != 0u) k2 = max(-64, min(64, 134 - static_cast<int>((amax >> 23) & 0xFF)));
            if (t == 0 && h + e < kGMax) qscale[(segc & 1u) * 8 + hh] = p.sm_scale_log2 * __uint_as_float(static_cast<uint32_t>(127 - k2) << 23);
            xs[e] = h + e < kGMax ? xq[hh] * __uint_as_float(static_cast<uint32_t>(k2 + 127) << 23) : 0.0f;
          }
          h2[h >> 1] = pack_f16x2(xs[0], xs[1]);    // exact: 8 significant bits, magnitude below 256
        }
        if (t < D) {
          const uint32_t col = (t >> 4) * 128 + (t & 15);
#pragma unroll
          for (int h = 0; h < kGMax; h += 2) {
            uint32_t v = h2[h >> 1];
            const uint32_t lead = e4m3_term(v, 1.0f);
            const uint32_t rest = f16x2_to_e4m3x2(v);
            if (h < G) { qb[col + h * 16] = static_cast<uint8_t>(lead & 0xFF); qb[kSboRows + col + h * 16] = static_cast<uint8_t>(rest & 0xFF); }
            if (h + 1 < G) { qb[col + (h + 1) * 16] = static_cast<uint8_t>(lead >> 8); qb[kSboRows + col + (h + 1) * 16] = static_cast<uint8_t>(rest >> 8); }
          }
        }
        bad = barrier_or(team_bar, kTeamThreads, bad);   // every thread has read the exchange words before the next query reuses them
        fence_proxy_async();
        mbar_arrive(&bar_qfull[segc & 1u]);
        // the raw buffer is free again: the rows of the segment two further on take its place
        if (t == 0 && si_next2 < nseg) fetch_q(plan.segs[si_next2], segc + 2);
      };

      // The piece of the segment before: its last product is folded in, and the piece handed to the
      // epilogue warp, behind the team's first tile of the next segment (flush_old), so that the end of a
      // segment does not wait for the tensor core.
      bool old_open = false, old_has_tile = false;
      uint32_t old_tile = 0, old_seg = 0;
      float o_old[kGMax], vref_old = 0.0f;
#pragma unroll
      for (int h = 0; h < kGMax; ++h) o_old[h] = 0.0f;
      auto flush_old = [&]() {
        bool ok = !bad;
        if (ok && old_has_tile) ok = wait_bar(&bar_empty[old_tile % C::kStages], (old_tile / C::kStages) & 1u, abort_flag);
        // the exchange area was last read by the epilogue warp for the segment before that one
        if (ok && old_seg >= 1) ok = wait_bar(&bar_efree[(old_seg - 1) & 1u], ((old_seg - 1) >> 1) & 1u, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        bad = bad || !ok;
        old_open = false;
        if (bad) return;
        if (old_has_tile) {
          uint32_t r[NP];
          tc_fence_after();
          const uint32_t obuf = tmem_o + NP * (old_tile & 3u) + lane_base;
#pragma unroll
          for (int half = 0; half < NP / 16; ++half) tmem_ld16_issue(obuf + half * 16, *reinterpret_cast<uint32_t(*)[16]>(&r[half * 16]));
#pragma unroll
          for (int half = 0; half < NP / 16; ++half) tmem_ld_wait(*reinterpret_cast<uint32_t(*)[16]>(&r[half * 16]));
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&bar_ofree[old_tile & 3u]);
#pragma unroll
          for (int h = 0; h < kGMax; ++h)
            o_old[h] += __uint_as_float(r[h]) + __uint_as_float(r[kGMax + h]) * 0.0625f + __uint_as_float(r[2 * kGMax + h]) * 0.00390625f;
        }
        float* xo = xch + team * C::kXchFloats;
#pragma unroll
        for (int h = 0; h < kGMax; ++h) xo[h * kTeamThreads + t] = o_old[h] * vref_old;
        mbar_arrive(&bar_efull[old_seg & 1u]);
      };

      if (team == 0 && nseg > 0) {
        if (t == 0) {
          fetch_q(plan.segs[0], seg_no);
          if (nseg > 1) fetch_q(plan.segs[1], seg_no + 1);
        }
        publish_q(seg_no, 2);
      }
      if (team == 1 && has_new) {
        // ---- Algorithm 1 phase 1 inside the step: the new token of every (sequence, kv head) whose last block
        // lies in this round.  Warp wq takes (tail segment, K | V) pairs wq, wq + 4, ..; the scale rule is the
        // write kernels' own (write_part), staged in a ring stage the copy warp has not reached yet.
        WriteParams wp;
        wp.cache = const_cast<uint8_t*>(p.cache);
        wp.k = p.k_new; wp.v = p.v_new;
        wp.slot_mapping = reinterpret_cast<const int64_t*>(p.slot_mapping);
        wp.token_stride = p.kv_token_stride;
        wp.num_tokens = B; wp.num_kv_heads = Hkv; wp.num_blocks = p.num_blocks;
        int task = 0;
        for (int si = 0; si < nseg; ++si) {
          const Segment& sg = plan.segs[si];
          if (!(sg.run_flags & kSegTail)) continue;
          for (int which = 0; which < 2; ++which, ++task) {
            if ((task & 3) != wq) continue;
            const long long slot = p.slot_mapping[sg.b];
            if (slot < 0) continue;                                          // Eq. 5: the token is skipped
            const long long blk = slot / kBlockSize;
            // the new token is the sequence's last position: its slot must name the last block of the table
            if (blk != plan.ids[sg.list_off + sg.n - 1] || static_cast<int>(slot % kBlockSize) != (sg.ctx_len - 1) % kBlockSize) {
              if (lane == 0) atomicCAS(p.status, 0, COOPT_ERR_INVALID_ARG);
            }
            if (blk >= p.num_blocks) continue;
            Group gr;
            gr.n = 1; gr.blk = static_cast<int>(blk); gr.tok[0] = sg.b; gr.off[0] = static_cast<int>(slot % kBlockSize);
            if (p.kv_e5m2) write_part<D, 1, true>(wp, gr, sg.g, which, write_stage + wq * (kBlockSize * D), lane);
            else write_part<D, 1, false>(wp, gr, sg.g, which, write_stage + wq * (kBlockSize * D), lane);
          }
        }
        // the granules are read next by the copy engine: order this warp's global (and staging) writes before it
        asm volatile("fence.proxy.async;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_wdone);
        COOPT_TRACE_CYCLES(p.trace, kTrWriteDone, t == 0);
      }
      for (int si = 0; si < nseg; ++si) {
        const Segment sg = plan.segs[si];
        const bool more = si + 1 < nseg;
        COOPT_TRACE_CYCLES(p.trace, kTrTeamSegBase + static_cast<int>(seg_no), tid == 0 && seg_no < 20);
        COOPT_TRACE_VALUE(p.trace, kTrSegTileBase + static_cast<int>(seg_no), tid == 0 && seg_no < 20, tile_no + 1);

        // the team's running softmax over its tiles of this segment
        float m_run[kGMax], l_run[kGMax], o_reg[kGMax];
#pragma unroll
        for (int h = 0; h < kGMax; ++h) { m_run[h] = -INFINITY; l_run[h] = 0.0f; o_reg[h] = 0.0f; }
        float vref = 0.0f;
        bool pending = false;       // a tile of this team whose P V product is not folded in yet
        bool q_due = team == 0 && more;   // the next segment's query is published behind this team's first tile
        uint32_t pend_tile = 0;

        // O_tile -> registers: o += term0 + term1 / 16 + term2 / 256 (o is kept on the scale of the tile being folded in)
        auto fold_issue = [&](uint32_t (&r)[NP]) {
          bool ok = !bad && wait_bar(&bar_empty[pend_tile % C::kStages], (pend_tile / C::kStages) & 1u, abort_flag);
          ok = __all_sync(0xffffffffu, ok);
          bad = bad || !ok;
          if (bad) return;
          tc_fence_after();
          const uint32_t obuf = tmem_o + NP * (pend_tile & 3u) + lane_base;
#pragma unroll
          for (int half = 0; half < NP / 16; ++half) tmem_ld16_issue(obuf + half * 16, *reinterpret_cast<uint32_t(*)[16]>(&r[half * 16]));
        };
        auto fold_finish = [&](uint32_t (&r)[NP]) {
          if (bad) return;
#pragma unroll
          for (int half = 0; half < NP / 16; ++half) tmem_ld_wait(*reinterpret_cast<uint32_t(*)[16]>(&r[half * 16]));
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&bar_ofree[pend_tile & 3u]);
#pragma unroll
          for (int h = 0; h < kGMax; ++h)
            o_reg[h] += (__uint_as_float(r[h]) + __uint_as_float(r[kGMax + h]) * 0.0625f +
                                               __uint_as_float(r[2 * kGMax + h]) * 0.00390625f);
          pending = false;
        };

        for (int k0 = 0; k0 < sg.n; k0 += kTileBlocks, ++tile_no) {
          if ((tile_no & 1u) != static_cast<uint32_t>(team)) continue;
          const int nb = min(kTileBlocks, sg.n - k0);
          const uint32_t stage = tile_no % C::kStages, buf = tile_no & 3u;
          uint8_t* st = ring + stage * C::kStageBytes;
          // scales of the granule that holds token t
          const float* hdr = reinterpret_cast<const float*>(st + C::kHdrOff + (t >> 4) * kFp8Header);
          const int tok0 = (sg.j0 + k0) * kBlockSize;
          const int ntok = min(nb * kBlockSize, sg.ctx_len - tok0);            // Eq. 9: tail of the context
          const uint32_t sbuf = tile_no & 3u;
          bool ok = !bad && wait_bar(&bar_sfull[sbuf], (tile_no >> 2) & 1u, abort_flag);
          ok = ok && wait_bar(&bar_full[stage], (tile_no / C::kStages) & 1u, abort_flag);
          ok = __all_sync(0xffffffffu, ok);
          bad = bad || !ok;
          float sc[kGMax];
          float sv = 0.0f;
          if (!bad) {
            tc_fence_after();
            uint32_t c[16];
            tmem_ld16_issue(tmem + 16 * sbuf + lane_base, c);
            const bool valid = t < ntok;
            const float sk = hdr[0];
            sv = valid ? hdr[1] : 0.0f;
            float qs[kGMax];
#pragma unroll
            for (int h = 0; h < kGMax; ++h) qs[h] = qscale[(seg_no & 1u) * 8 + h] * sk;
            tmem_ld_wait(c);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bar_sfree[sbuf]);
            int* rw = my_red_max + wq * 12;
#pragma unroll
            for (int h = 0; h < kGMax; ++h) {
              sc[h] = valid ? (__uint_as_float(c[h]) + __uint_as_float(c[8 + h])) * qs[h] : -INFINITY;
              const int wm = __reduce_max_sync(0xffffffffu, f32_to_ordered(sc[h]));
              if (lane == 0) rw[h] = wm;
            }
            const int wv = __reduce_max_sync(0xffffffffu, __float_as_int(sv));     // V scales are non-negative
            if (lane == 0) rw[8] = wv;
          }
          bad = barrier_or(team_bar, kTeamThreads, bad);
          if (bad) { team_bad = true; break; }
          const int* rmx = my_red_max;
          // reference V scale: the largest met so far by the team in the segment (uniform over the team)
          const float vmax = __int_as_float(max(max(rmx[8], rmx[20]), max(rmx[32], rmx[44])));
          const float vnew = fmaxf(vref, vmax);
          const float vr = vnew > vref ? __fdividef(vref, vnew) : 1.0f;
          const float pvs = vnew > 0.0f ? __fdividef(sv, vnew) * 256.0f : 0.0f;   // probabilities are carried times 2^8
          vref = vnew;
          float a_o[kGMax], pw[kGMax];
#pragma unroll
          for (int h = 0; h < kGMax; ++h) {
            const float m_tile = ordered_to_f32(max(max(rmx[h], rmx[12 + h]), max(rmx[24 + h], rmx[36 + h])));
            const float m_new = fmaxf(m_run[h], m_tile);
            const float mu = m_new == -INFINITY ? 0.0f : m_new;
            const float a_m = ex2(m_run[h] - mu);
            const float pr = ex2(sc[h] - mu);
            l_run[h] = l_run[h] * a_m + pr;
            m_run[h] = m_new;
            a_o[h] = a_m * vr;
            pw[h] = pr * pvs;
          }
          // ---- probabilities of token t: three E4M3 terms per head, one byte per row of Pg ----------
          {
            uint8_t* pb = pbuf + buf * C::kPBytes + (t >> 4) * 128 + (t & 15);
#pragma unroll
            for (int h = 0; h < kGMax; h += 2) {
              uint32_t v = pack_f16x2(pw[h], h + 1 < kGMax ? pw[h + 1] : 0.0f);
#pragma unroll
              for (int term = 0; term < 3; ++term) {
                const uint32_t codes = term < 2 ? e4m3_term(v, 16.0f) : f16x2_to_e4m3x2(v);
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
            // an odd number of blocks: the last instruction also reads the slot behind them
            if ((nb & 1) != 0 && t < D)
              *reinterpret_cast<uint4*>(st + C::kKArea + nb * C::kPart + (t >> 3) * 128 + (t & 7) * 16) = make_uint4(0u, 0u, 0u, 0u);
            fence_proxy_async();
            mbar_arrive(&bar_pfull[buf]);
            COOPT_TRACE_CYCLES(p.trace, kTrFirstProbs, tid == 0 && tile_no == 0);
            COOPT_TRACE_CYCLES(p.trace, kTrProbsTileBase + static_cast<int>(tile_no), t == 0 && tile_no < 32);
          }
          // the product of the team's previous tile (its own buffers, so nothing above had to wait for it)
          if (pending) {
            uint32_t o_raw[NP];
            fold_issue(o_raw);
            fold_finish(o_raw);
          }
#pragma unroll
          for (int h = 0; h < kGMax; ++h) o_reg[h] *= a_o[h];      // what is folded in so far, on the scale of this tile's product
          pending = true;
          pend_tile = tile_no;
          if (q_due) { publish_q(seg_no + 1, si + 3); q_due = false; }
          if (old_open) flush_old();
        }
        // (a team whose wait ran out keeps company until the next barrier makes it known to everybody)
        if (q_due) publish_q(seg_no + 1, si + 3);   // the segment had no tile for this team

        // ---- end of segment: the team's sums and maxima go to the epilogue warp now, its output follows
        // once the last product has been folded in (flush_old, behind the next segment's first tile)
        if (team_bad) break;
        if (old_open) flush_old();            // the segment gave this team no tile
        {
          // (the area of this parity was last read for segment seg_no - 2, which the flush of segment
          // seg_no - 1 has waited for)
          float* mls = mlbuf + ((seg_no & 1u) * 2 + team) * C::kMlFloats;
#pragma unroll
          for (int h = 0; h < kGMax; ++h) {
            const float ws = warp_sum(l_run[h]);
            if (lane == 0) mls[wq * 8 + h] = ws;
            if (t == 0) mls[32 + h] = m_run[h];
          }
        }
        old_open = true;
        old_has_tile = pending;
        old_tile = pend_tile;
        old_seg = seg_no;
        vref_old = vref;
#pragma unroll
        for (int h = 0; h < kGMax; ++h) o_old[h] = pending ? o_reg[h] : 0.0f;
        ++seg_no;
      }
      if (old_open) flush_old();              // the round's last segment
      COOPT_TRACE_CYCLES(p.trace, kTrTeamsDone, tid == 0);
      if (bad && t == 0) atomicCAS(p.status, 0, COOPT_ERR_TIMEOUT);
    }

    __syncthreads();
    if (*abort_flag != 0 || last_round) break;
    // roles that skipped their counters (idle lanes) are not using them; the others agree by construction
    plan_at += round_bytes;
    ++round_no;
    if (tid == 0) {
      fence_proxy_async();                      // the round just read gives way to the next one
      mbar_expect_tx(bar_plan, kPlanFirstChunk);
      bulk_copy_g2s(plan_smem, plan_region + plan_at, kPlanFirstChunk, bar_plan);
    }
  }
  COOPT_TRACE_CYCLES(p.trace, kTrExit, tid == 0);
  COOPT_TRACE_NS(p.trace, kTrExitNs, tid == 0);

  // ---- exit: copies still in flight get a bounded time to land, tensor memory is returned -----------
  if (*abort_flag != 0 && warp == kProducerWarp && lane == 0) {
    for (uint32_t s = 0; s < static_cast<uint32_t>(C::kStages) && s < tile_no; ++s) {
      const uint32_t last = tile_no - 1 - s;        // the last tile issued into stage last % kStages
      mbar_wait_bounded(&bar_full[last % C::kStages], (last / C::kStages) & 1u);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(C::kTmemCols) : "memory");
}

// The copy engine's two views of a cache (parts, headers), encoded once per (cache, shape, device) and kept:
// a serving loop launches on the same few caches over and over.
struct CacheMaps {
  const void* data;
  long long granules;
  int gran, part, dev;
  CUtensorMap map_part, map_hdr;
};
bool cache_maps(const void* data, long long granules, int gran, int part, CUtensorMap* map_part, CUtensorMap* map_hdr) {
  static std::mutex mu;
  static std::vector<CacheMaps> known;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return false;
  std::lock_guard<std::mutex> lock(mu);
  for (const CacheMaps& m : known) {
    if (m.data == data && m.granules == granules && m.gran == gran && m.part == part && m.dev == dev) {
      *map_part = m.map_part; *map_hdr = m.map_hdr;
      return true;
    }
  }
  CacheMaps m;
  m.data = data; m.granules = granules; m.gran = gran; m.part = part; m.dev = dev;
  if (!encode_cache_map(&m.map_part, data, granules, gran, part / 8) || !encode_cache_map(&m.map_hdr, data, granules, gran, kFp8Header / 8))
    return false;
  if (known.size() >= 256) known.erase(known.begin());
  known.push_back(m);
  *map_part = m.map_part; *map_hdr = m.map_hdr;
  return true;
}

template <int D, int NP>
int launch_umma_one(DecodeParams p, int grid, bool overlap_previous, cudaStream_t stream) {
  using C = UCfg<D, NP>;
  CUtensorMap map_part, map_hdr;
  const long long granules = static_cast<long long>(p.num_blocks) * p.num_kv_heads;
  if (!cache_maps(p.cache, granules, C::kGran, C::kPart, &map_part, &map_hdr)) return COOPT_ERR_CUDA;
  if (!configure_kernel_smem(reinterpret_cast<const void*>(&paged_decode_umma_kernel<D, NP>), C::kSmemBytes)) return COOPT_ERR_CUDA;
#ifdef COOPT_TRACE
  p.trace = trace_buffer();
  p.plan_rotate = trace_plan_rotate();
#endif
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(grid));
  cfg.blockDim = dim3(kUmmaThreads);
  cfg.dynamicSmemBytes = C::kSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = overlap_previous ? 1 : 0;     // the kernel may then start while the one before it still runs
  return cudaLaunchKernelEx(&cfg, paged_decode_umma_kernel<D, NP>, p, map_part, map_hdr) == cudaSuccess ? COOPT_OK : COOPT_ERR_CUDA;
}

}  // namespace

// FP8 cache: group sizes 1..5 use 16 probability rows, 6..8 use 32.
int launch_paged_decode_umma(const DecodeParams& p, int head_dim, int grid, bool overlap_previous, cudaStream_t stream) {
  if (p.group <= 5)
    return head_dim == 128 ? launch_umma_one<128, 16>(p, grid, overlap_previous, stream) : launch_umma_one<64, 16>(p, grid, overlap_previous, stream);
  return head_dim == 128 ? launch_umma_one<128, 32>(p, grid, overlap_previous, stream) : launch_umma_one<64, 32>(p, grid, overlap_previous, stream);
}

}  // namespace coopt
