// Chunked prefill against the paged FP8 cache on the 5th-generation tensor cores (head_dim 128): Eq. 1
// with the causal K_{<=t}, Eq. 6 dequantisation on load, Eq. 7-8 grouped-query sharing, Eq. 9 valid
// blocks only, Eq. 10 max-subtracted softmax, for runs of several query tokens per sequence.
//
// A CTA owns one (sequence, kv head, tile of consecutive query tokens).  Its 128 rows are the (query
// token, query head of the group) pairs of the tile, so the K/V stream of the kv head is fetched once
// for all G heads (Algorithm 2).  The E4M3 codes of the cache feed tcgen05.mma kind::f8f6f4 as they are:
//     S [128 rows x 128 keys] = Q  [128 x D] . Ktile^T      kind::f8f6f4: Q as two exact E4M3 terms of the bf16 query
//     O [128 rows x D]       += P  [128 x 128 keys] . Vtile  kind::f16: P rounded once to f16, the V codes widened to f16 (exact)
// with fp32 accumulators in tensor memory.  The K scale of a block multiplies the logits of its 16 keys,
// the V scale is folded into the probabilities.  (Carrying P as E4M3 terms instead, three per probability for
// the same 11 bits, kept the V codes as they are but cost five conversions per pair of probabilities on the
// SM's conversion pipe, which then bounded the kernel; widening V costs one conversion per pair of codes and
// a tile of V is a sixteenth of a tile of P per query row.)
//
// The context is walked twice, 128 keys (eight cache blocks) at a time.  The first walk fetches K only and
// leaves every row's maximum logit (and the largest V scale); the second recomputes the logits, so every
// probability is exp(s - final maximum) <= 1 and the output accumulator in tensor memory is never
// rescaled.  The second product over K costs a third more tensor work and K traffic (out of L2), and
// removes the read-modify-write of 128 x 128 accumulators whenever a maximum moves.
//
// Warp roles (608 threads):
//   warps 0-7, 8-15  two softmax teams, even and odd tiles.  Two threads of a team share row r: warps 0-3 of
//               the team take the tile's first four cache blocks, warps 4-7 the last four; a thread reads its
//               row's logits from tensor memory 16 at a time (one cache block: one pair of scales), and
//               maxima and sums are exchanged only at the end of a walk;
//   warp 16     copies: gather requests over the tensor map of the cache (K parts, V parts, headers of
//               four granules each) into four slots of 16 KB + 256 B.  The first walk uses all four for K
//               tiles (and their scales); in the second walk two take K tiles, freed as soon as the logits
//               are computed, and two take V tiles and the scales, freed as soon as the tile's team has widened
//               the codes into its f16 operand;
//   warp 17     one lane issues the S instructions; warp 18 one lane issues the P V instructions.
// Every wait is bounded; a wait that runs out is reported in the status word and all roles leave through
// the common exit, which frees the tensor memory.
#include "coopt_umma.cuh"

namespace coopt {

namespace {

constexpr int kPuRows = 128;                               // rows of a tile = threads of half a team
constexpr int kPuTeam = 2 * kPuRows;                       // eight warps: four tensor-memory lane quarters x two halves of the columns
constexpr int kPuSm = 2 * kPuTeam;                         // warps 0-15
constexpr int kPuProducer = 16, kPuSWarp = 17, kPuPvWarp = 18;
constexpr int kPuThreads = 608;
constexpr int kPuTileBlocks = 8;
constexpr int kPuTileKeys = kPuTileBlocks * kBlockSize;   // 128
constexpr int kPuD = 128;
constexpr int kPuSlots = 4;                                // of the copy ring
constexpr int kPuKSlots = 2, kPuVSlots = 2;               // second walk: slots 0-1 take K tiles, slots 2-3 V tiles and scales
constexpr float kPuLog2e = 1.4426950408889634f;
constexpr float kPuGain = 256.0f;                          // probabilities are carried times 2^8 (at most 256 < 448)

struct PrefillUmmaParams {
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
  int kv_e5m2;             // the cache codes are E5M2 (the format ablation)
  float sm_scale_log2;
  int* status;
};

struct PuCfg {
  static constexpr int kPart = kBlockSize * kPuD;                 // 2048: K (or V) codes of one granule
  static constexpr int kGran = granule_bytes(kPuD, true);
  static constexpr int kKArea = kPuTileBlocks * kPart;            // 16 KB: the K parts, or the V parts, of a tile
  static constexpr int kHdrOff = kKArea;                          // behind them the eight headers (scales) of the tile
  static constexpr int kSlot = kHdrOff + kPuTileBlocks * kFp8Header;   // 16,640
  static constexpr int kOperand = 128 * 128;                      // one 128 x 128 operand of codes
  static constexpr int kRingOff = 0;
  static constexpr int kQOff = kRingOff + kPuSlots * kSlot;          // Q: lead term, remainder term
  static constexpr int kOperand16 = 128 * 128 * 2;                   // one 128 x 128 operand of f16 values
  static constexpr int kPOff = kQOff + 2 * kOperand;                 // P: [team], f16
  static constexpr int kV16Off = kPOff + 2 * kOperand16;             // V^T of a tile widened to f16: [team]
  static constexpr int kBarOff = kV16Off + 2 * kOperand16;
  static constexpr int kNumBars = 2 * kPuSlots + kPuKSlots + 2 * kPuVSlots + 2 + 2 + 2;   // full, free1, kdone, vdone, vread, sfull, sfree, pfull
  static constexpr int kMiscOff = kBarOff + kNumBars * 8;
  static constexpr int kSmemBytes = kMiscOff + 64;
  static_assert(kSlot % 128 == 0 && kSmemBytes <= 232448, "shared memory of one CTA");
};

__global__ void __launch_bounds__(kPuThreads, 1) paged_prefill_umma_kernel(const PrefillUmmaParams p, const __grid_constant__ CUtensorMap map_part,
                                                                          const __grid_constant__ CUtensorMap map_hdr) {
  using C = PuCfg;
  constexpr int D = kPuD;
  extern __shared__ __align__(128) uint8_t smem[];
  uint8_t* ring = smem + C::kRingOff;
  uint8_t* qbuf = smem + C::kQOff;
  uint8_t* pbuf = smem + C::kPOff;
  uint8_t* v16buf = smem + C::kV16Off;
  // float [4 parts of a row][128] maxima and [4][128] sums share the probability operands' memory: the maxima are
  // exchanged before the first probability is written, the sums after the last P V instruction has finished
  float* xch = reinterpret_cast<float*>(smem + C::kPOff);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::kBarOff);
  // Every signal that frees a slot is per slot: its next phase cannot complete before the slot has been
  // refilled, so the parity a waiter looks for is never overtaken.
  uint64_t* bar_full = bars;                         // [kPuSlots] the copies into the slot have landed
  uint64_t* bar_free1 = bar_full + kPuSlots;         // [kPuSlots] first walk: the tile's team has read its logits and scales
  uint64_t* bar_kdone = bar_free1 + kPuSlots;        // [kPuKSlots] second walk: the logits of the K tile in the slot are computed
  uint64_t* bar_vdone = bar_kdone + kPuKSlots;       // [kPuVSlots] second walk: the P V instructions of the V tile in the slot are done
  uint64_t* bar_vread = bar_vdone + kPuVSlots;       // [kPuVSlots] second walk: the tile's team has widened the V tile in the slot
  uint64_t* bar_sfull = bar_vread + kPuVSlots;       // [2] logits of a tile are in tensor memory (buffer = tile & 1 = team)
  uint64_t* bar_sfree = bar_sfull + 2;               // [2] the team's eight warps have read them (and the tile's scales)
  uint64_t* bar_pfull = bar_sfree + 2;               // [2] the team's probabilities of a tile are in shared memory
  int* misc = reinterpret_cast<int*>(smem + C::kMiscOff);   // [0] sequence, [1] first query, [2] abort flag, [3] tensor memory, [4..7] V scale maxima
  volatile int* abort_flag = misc + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(misc + 3);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
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
    *abort_flag = 0;
    for (int i = 0; i < kPuSlots; ++i) { mbar_init(&bar_full[i], 1); mbar_init(&bar_free1[i], 8); }
    for (int i = 0; i < kPuKSlots; ++i) mbar_init(&bar_kdone[i], 1);
    for (int i = 0; i < kPuVSlots; ++i) { mbar_init(&bar_vdone[i], 1); mbar_init(&bar_vread[i], 8); }
    for (int i = 0; i < 2; ++i) { mbar_init(&bar_sfull[i], 1); mbar_init(&bar_sfree[i], 8); mbar_init(&bar_pfull[i], kPuTeam); }
    mbar_fence_init();
  }
  if (tid == kPuProducer * 32) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_part) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_hdr) : "memory");
  }
  __syncthreads();
  const int b = misc[0];
  if (b < 0) return;                                 // uniform over the CTA: nothing has been allocated yet
  const int q0 = misc[1];
  const int row_base = p.cu_q_lens[b];
  const int n_new = p.cu_q_lens[b + 1] - row_base;
  const int nq = min(TQ, n_new - q0);
  const int L = max(0, min(p.context_lens[b], p.max_blocks_per_seq * kBlockSize));
  // last position any row of the tile may see (Eq. 1: K_{<=t})
  const int kv_end = p.causal ? max(0, min(L, L - n_new + q0 + nq)) : L;
  const int n_tiles = (kv_end + kPuTileKeys - 1) / kPuTileKeys;
  const int n_blocks = (kv_end + kBlockSize - 1) / kBlockSize;

  // ---- this thread's row (softmax teams: row r belongs to the two threads r and r + 128 of either team) ---
  const int r = tid & (kPuRows - 1);
  const int half = (tid >> 7) & 1;                    // which four cache blocks of a tile
  const int qi = r / G;
  const bool live = tid < kPuSm && qi < nq;
  const size_t grow = static_cast<size_t>(row_base + q0 + (live ? qi : 0)) * Hq + g * G + (live ? r % G : 0);
  // index of the last visible key of the row; -1 hides everything
  const int lim = live ? (p.causal ? min(L - 1, L - n_new + q0 + qi) : L - 1) : -1;

  if (n_tiles == 0) {
    // nothing visible: all-zero rows
    if (tid < kPuRows && live)
      for (int d = 0; d < D; d += 8) *reinterpret_cast<uint4*>(p.out + grow * D + d) = make_uint4(0u, 0u, 0u, 0u);
    return;
  }

  // ---- set-up: tensor memory, the query operand ---------------------------------------
  if (warp == kPuSWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // Row r of the query operand: the bf16 row scaled by a power of two into [128, 256) (undone on the
  // logits) is the exact sum of its nearest E4M3 value and the E4M3 value of the remainder.  Element
  // (row, byte k) of an operand sits at (row / 8) * 1024 + (k / 16) * 128 + (row % 8) * 16 + k % 16.
  float qscale = 0.0f;       // logits of this row = tensor-memory value * qscale * K scale of the block
  if (tid < kPuSm) {
    // every thread of the teams needs its row's scale; threads 0..127 also build the operand
    uint32_t amax = 0;
    if (live) {
#pragma unroll 4
      for (int c = 0; c < D / 8; ++c) {
        const uint4 v = *reinterpret_cast<const uint4*>(p.q + grow * D + c * 8);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) amax = max(amax, max((w[e] << 16) & 0x7FFFFFFFu, w[e] & 0x7FFF0000u));   // |bf16| as fp32 bits
      }
    }
    int k2 = 0;
    if (amax != 0u) k2 = max(-64, min(64, 134 - static_cast<int>((amax >> 23) & 0xFF)));
    qscale = p.sm_scale_log2 * __uint_as_float(static_cast<uint32_t>(127 - k2) << 23);
    if (tid < kPuRows) {
      const float up = __uint_as_float(static_cast<uint32_t>(k2 + 127) << 23);
      uint8_t* qrow = qbuf + (r >> 3) * 1024 + (r & 7) * 16;
#pragma unroll 2
      for (int c = 0; c < D / 16; ++c) {            // 16 elements = one 16-byte chunk of each term
        uint4 raw[2];
#pragma unroll
        for (int k = 0; k < 2; ++k) raw[k] = live ? *reinterpret_cast<const uint4*>(p.q + grow * D + c * 16 + k * 8) : make_uint4(0u, 0u, 0u, 0u);
        uint32_t lead[4], rest[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {               // four elements = two packed pairs
          const uint4 v = raw[e >> 1];
          const uint32_t w0 = (e & 1) ? v.z : v.x, w1 = (e & 1) ? v.w : v.y;
          uint32_t h0 = pack_f16x2(__uint_as_float(w0 << 16) * up, __uint_as_float(w0 & 0xFFFF0000u) * up);
          uint32_t h1 = pack_f16x2(__uint_as_float(w1 << 16) * up, __uint_as_float(w1 & 0xFFFF0000u) * up);
          const uint32_t l0 = e4m3_term(h0, 1.0f), l1 = e4m3_term(h1, 1.0f);
          lead[e] = l0 | (l1 << 16);
          rest[e] = f16x2_to_e4m3x2(h0) | (f16x2_to_e4m3x2(h1) << 16);
        }
        *reinterpret_cast<uint4*>(qrow + c * 128) = make_uint4(lead[0], lead[1], lead[2], lead[3]);
        *reinterpret_cast<uint4*>(qrow + C::kOperand + c * 128) = make_uint4(rest[0], rest[1], rest[2], rest[3]);
      }
    }
  }
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tmem_o = tmem + 256;                 // logits buffer b at column 128 b, output at 256
  const uint32_t lane_base = static_cast<uint32_t>(warp & 3) * 32u << 16;
  const int total = 2 * n_tiles;                      // tiles of both walks, numbered in order of use
  // Slots and the phase of a slot's "landed" barrier.  First walk: tile T lands in slot T % 6 (its use
  // T / 6 of that slot).  Second walk: the K parts of tile t land in slot t % 2 (use t / 2 after the slot's
  // first-walk uses), its V parts and scales in slot 2 + t % 4 (use t / 4 after the first-walk uses).
  auto uses1 = [&](int slot) { return n_tiles > slot ? (n_tiles - slot + kPuSlots - 1) / kPuSlots : 0; };
  auto kslot_par = [&](int t) { return static_cast<uint32_t>(uses1(t % kPuKSlots) + t / kPuKSlots) & 1u; };
  auto vslot_par = [&](int t) { return static_cast<uint32_t>(uses1(kPuKSlots + t % kPuVSlots) + t / kPuVSlots) & 1u; };
  uint32_t pend_mask = 0, pend_par = 0;               // copy lane: the latest phase expected of every slot it has filled

  if (warp == kPuProducer) {
    // ================= copies: first walk K parts and headers, second walk V parts as well ================
    // Lane 3 q + w (q = 0, 1; w = 0, 1, 2) fetches the K parts (w = 0), the V parts (w = 1) or the headers
    // (w = 2) of granules 4 q .. 4 q + 3 of the tile.  Rows past the last block repeat the tile's first one.
    bool ok = true;
    const int q4 = lane / 3, what = lane - 3 * q4;
    const int x = what * (C::kPart / 8);
    const uint32_t dst_off = what == 2 ? C::kHdrOff + q4 * 4 * kFp8Header : q4 * 4 * C::kPart;       // inside the slot
    const CUtensorMap* map = what == 2 ? &map_hdr : &map_part;
    // The physical blocks are looked up 32 at a time (four tiles, one per lane), a batch ahead of their use, so
    // that the copy lane never waits for the block table (range-checked: a bad id is reported in the status
    // word and replaced by block 0, never dereferenced).  Batches are numbered through both walks.
    const int* trow = p.block_table + static_cast<size_t>(b) * p.max_blocks_per_seq;
    const int nbatch = (n_tiles + 3) / 4;
    auto load_batch = [&](int lb) -> int {
      if (lb >= 2 * nbatch) return 0;
      const int j = (lb >= nbatch ? lb - nbatch : lb) * 32 + lane;
      int id = j < n_blocks ? trow[j] : 0;
      if (id < 0 || id >= p.num_blocks) { atomicCAS(p.status, 0, COOPT_ERR_INVALID_ARG); id = 0; }
      return id;
    };
    int cur_lb = 0;
    int ids_cur = load_batch(0), ids_next = load_batch(1);
    for (int T = 0; T < total; ++T) {
      const bool second = T >= n_tiles;
      const int t = second ? T - n_tiles : T;
      const int nb = min(kPuTileBlocks, n_blocks - t * kPuTileBlocks);
      const int ngroups = (nb + 3) / 4;
      const int lb = (second ? nbatch : 0) + (t >> 2);
      if (lb != cur_lb) { ids_cur = ids_next; cur_lb = lb; ids_next = load_batch(lb + 1); }
      int rows[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int j = (q4 & 1) * 4 + i;                             // block of the tile (lanes past the six copy lanes fetch along)
        rows[i] = __shfl_sync(0xffffffffu, ids_cur, (t & 3) * 8 + (j < nb ? j : 0)) * Hkv + g;
      }
      if (!second) {
        const int slot = T % kPuSlots;
        if (lane == 0) {
          if (T >= kPuSlots) ok = wait_bar(&bar_free1[slot], static_cast<uint32_t>(T / kPuSlots - 1) & 1u, abort_flag);
          if (ok) {
            mbar_expect_tx(&bar_full[slot], ngroups * 4 * (C::kPart + kFp8Header));
            pend_mask |= 1u << slot;
            pend_par = (pend_par & ~(1u << slot)) | ((static_cast<uint32_t>(T / kPuSlots) & 1u) << slot);
          }
        }
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) break;
        if (lane < 3 * ngroups && what != 1)
          gather4_g2s(ring + slot * C::kSlot + dst_off, map, x, rows[0], rows[1], rows[2], rows[3], &bar_full[slot]);
      } else {
        const int ks = t % kPuKSlots, vq = t % kPuVSlots, vs = kPuKSlots + vq;
        if (lane == 0) {
          // who used the slots before: the second walk's tile two (K) or four (V) back, else the slot's last tile of the first walk
          if (t >= kPuKSlots) ok = wait_bar(&bar_kdone[ks], static_cast<uint32_t>(t / kPuKSlots - 1) & 1u, abort_flag);
          else if (uses1(ks) > 0) ok = wait_bar(&bar_free1[ks], static_cast<uint32_t>(uses1(ks) - 1) & 1u, abort_flag);
          if (ok) {
            if (t >= kPuVSlots) ok = wait_bar(&bar_vread[vq], static_cast<uint32_t>(t / kPuVSlots - 1) & 1u, abort_flag);
            else if (uses1(vs) > 0) ok = wait_bar(&bar_free1[vs], static_cast<uint32_t>(uses1(vs) - 1) & 1u, abort_flag);
          }
          if (ok) {
            mbar_expect_tx(&bar_full[ks], ngroups * 4 * C::kPart);
            mbar_expect_tx(&bar_full[vs], ngroups * 4 * (C::kPart + kFp8Header));
            pend_mask |= (1u << ks) | (1u << vs);
            pend_par = (pend_par & ~((1u << ks) | (1u << vs))) | (kslot_par(t) << ks) | (vslot_par(t) << vs);
          }
        }
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) break;
        if (lane < 3 * ngroups) {
          const int slot = what == 0 ? ks : vs;
          gather4_g2s(ring + slot * C::kSlot + dst_off, map, x, rows[0], rows[1], rows[2], rows[3], &bar_full[slot]);
        }
      }
    }
    if (!ok && lane == 0) atomicCAS(p.status, 0, COOPT_ERR_TIMEOUT);
  } else if (warp == kPuSWarp) {
    // ================= logits: S = Q . Ktile^T, both terms of Q (one lane) ====================================
    if (lane == 0) {
      bool ok = true;
      const uint64_t desc_k = umma_desc(smem_u32(ring), 128, 8 * D), desc_q = umma_desc(smem_u32(qbuf), 128, 1024);
      for (int T = 0; T < total && ok; ++T) {
        const uint32_t buf = T & 1u, use = T >> 1;
        const bool second = T >= n_tiles;
        const int t = second ? T - n_tiles : T;
        const uint32_t slot = second ? t % kPuKSlots : T % kPuSlots;
        ok = wait_bar(&bar_full[slot], second ? kslot_par(t) : static_cast<uint32_t>(T / kPuSlots) & 1u, abort_flag);
        if (ok && use > 0) ok = wait_bar(&bar_sfree[buf], (use - 1) & 1u, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint64_t dk = desc_k + ((slot * C::kSlot) >> 4);
#pragma unroll
        for (int term = 0; term < 2; ++term)
#pragma unroll
          for (int ks = 0; ks < D / 32; ++ks)
            umma_f8(tmem + 128 * buf, desc_q + ((term * C::kOperand) >> 4) + ks * 16, dk + ks * 16, umma_idesc(128, 0, p.kv_e5m2), (term | ks) != 0);
        umma_commit(&bar_sfull[buf]);
      }
      if (!ok) atomicCAS(p.status, 0, COOPT_ERR_TIMEOUT);
    }
  } else if (warp == kPuPvWarp) {
    // ================= outputs: O += P . Vtile, both terms of P (one lane) ===================================
    if (lane == 0) {
      bool ok = true;
      // both operands of P V are f16, K-major: 8 rows x 16 bytes (8 values) per core matrix, cores of a row group 128 bytes
      // apart along the keys, row groups 2048 bytes apart
      const uint64_t desc_v = umma_desc(smem_u32(v16buf), 128, 2048), desc_p = umma_desc(smem_u32(pbuf), 128, 2048);
      for (int T = n_tiles; T < total && ok; ++T) {
        const int t = T - n_tiles;
        const uint32_t vq = t % kPuVSlots, team = T & 1u;
        // the team's tiles of the second walk so far
        const int first = n_tiles + ((static_cast<int>(team) - n_tiles % 2) + 2) % 2;
        const uint32_t use = (T - first) >> 1;
        ok = wait_bar(&bar_pfull[team], use & 1u, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const int nb = min(kPuTileBlocks, n_blocks - t * kPuTileBlocks);      // 16 keys (one cache block) per instruction
        const uint64_t dv = desc_v + ((team * C::kOperand16) >> 4), dp = desc_p + ((team * C::kOperand16) >> 4);
        for (int ks = 0; ks < nb; ++ks) umma_f16(tmem_o, dp + ks * 16, dv + ks * 16, umma_idesc(D), (t | ks) != 0);
        umma_commit(&bar_vdone[vq]);        // the team's two f16 operands are free again
      }
      if (!ok) atomicCAS(p.status, 0, COOPT_ERR_TIMEOUT);
    }
  } else {
    // ================= softmax teams ================================================================================
    const int team = warp >> 3;
    const int c_lo = half * (kPuTileBlocks / 2), c_hi = c_lo + kPuTileBlocks / 2;   // this thread's cache blocks of a tile
    bool bad = false;
    float m_row = -INFINITY, l_row = 0.0f, v_max = 0.0f;
    uint8_t* prow = pbuf + team * C::kOperand16 + (r >> 3) * 2048 + (r & 7) * 16;      // row r of the team's P operand
    uint8_t* vrow = v16buf + team * C::kOperand16 + (r >> 3) * 2048 + (r & 7) * 16;    // dim r of the team's V^T operand

    // ---- first walk: the row's maximum logit, and the largest V scale ------------------------------------
    for (int T = team; T < n_tiles; T += 2) {
      const uint32_t slot = T % kPuSlots, buf = T & 1u;
      const uint8_t* st = ring + slot * C::kSlot;
      bool ok = !bad && wait_bar(&bar_full[slot], static_cast<uint32_t>(T / kPuSlots) & 1u, abort_flag);
      ok = ok && wait_bar(&bar_sfull[buf], (T >> 1) & 1u, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      bad = bad || !ok;
      if (bad) break;
      tc_fence_after();
      const int key0 = T * kPuTileKeys;
      const int nkeys = min(kPuTileKeys, kv_end - key0);
#pragma unroll 2
      for (int c = c_lo; c < c_hi; ++c) {
        if (c * kBlockSize >= nkeys) break;                       // uniform over the warp
        uint32_t s[16];
        tmem_ld16_issue(tmem + 128 * buf + 16 * c + lane_base, s);
        const float* hdr = reinterpret_cast<const float*>(st + C::kHdrOff + c * kFp8Header);
        const float sk = hdr[0] * qscale;
        v_max = fmaxf(v_max, hdr[1]);
        const int visible = lim - (key0 + c * kBlockSize);         // keys 0 .. visible of this block are seen by the row
        tmem_ld_wait(s);
#pragma unroll
        for (int j = 0; j < 16; ++j)
          if (j <= visible) m_row = fmaxf(m_row, __uint_as_float(s[j]) * sk);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) { mbar_arrive(&bar_sfree[buf]); mbar_arrive(&bar_free1[slot]); }
    }
    // the maxima of the four threads that saw part of row r (two teams x two halves of the columns)
    const int part = team * 2 + half;
    xch[part * kPuRows + r] = m_row;
    if (r == 0) reinterpret_cast<float*>(misc + 4)[part] = v_max;
    bad = barrier_or(1, kPuSm, bad);
    if (!bad) {
      m_row = fmaxf(fmaxf(xch[r], xch[kPuRows + r]), fmaxf(xch[2 * kPuRows + r], xch[3 * kPuRows + r]));
      const float* vm = reinterpret_cast<const float*>(misc + 4);
      v_max = fmaxf(fmaxf(vm[0], vm[1]), fmaxf(vm[2], vm[3]));
    }
    bad = barrier_or(1, kPuSm, bad);          // everybody has read the maxima: their memory may take probabilities
    const float m_use = m_row == -INFINITY ? 0.0f : m_row;
    const float v_inv = v_max > 0.0f ? kPuGain / v_max : 0.0f;

    // ---- second walk: probabilities against the final maximum (f16), the V tile widened to f16 -----------
    int mine = 0;                                                  // this team's tiles of the second walk so far
    for (int T = n_tiles + ((team - n_tiles % 2) + 2) % 2; T < total && !bad; T += 2, ++mine) {
      const int t = T - n_tiles;
      const uint32_t vq = t % kPuVSlots, buf = T & 1u;
      const uint8_t* st = ring + (kPuKSlots + vq) * C::kSlot;      // the tile's V parts, and behind them its scales
      bool ok = wait_bar(&bar_full[kPuKSlots + vq], vslot_par(t), abort_flag);
      ok = ok && wait_bar(&bar_sfull[buf], (T >> 1) & 1u, abort_flag);
      // the logits are computed: the tile's K slot can be refilled
      if (ok && (warp & 7) == 0 && lane == 0) mbar_arrive(&bar_kdone[t % kPuKSlots]);
      // the team's previous tile must have left the probability operand
      if (ok && mine > 0) ok = wait_bar(&bar_vdone[(t - 2) % kPuVSlots], static_cast<uint32_t>((t - 2) / kPuVSlots) & 1u, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      bad = bad || !ok;
      if (bad) break;
      tc_fence_after();
      const int key0 = t * kPuTileKeys;
      const int nkeys = min(kPuTileKeys, kv_end - key0);
      const int nb = (nkeys + kBlockSize - 1) / kBlockSize;
#pragma unroll 2
      for (int c = c_lo; c < c_hi; ++c) {
        if (c >= nb) break;                               // uniform over the warp: the P V instructions stop at block nb
        uint32_t s[16];
        tmem_ld16_issue(tmem + 128 * buf + 16 * c + lane_base, s);
        const float* hdr = reinterpret_cast<const float*>(st + C::kHdrOff + c * kFp8Header);
        const float sk = hdr[0] * qscale;
        const float pv = hdr[1] * v_inv;
        const int visible = lim - (key0 + c * kBlockSize);
        // dim r of V^T, the 16 tokens of block c: widened to f16 (exact) while the logits are on their way
        const uint4 vc = *reinterpret_cast<const uint4*>(st + c * C::kPart + (r >> 3) * 128 + (r & 7) * 16);
        const int keep = nkeys - c * kBlockSize;          // tokens of the block inside the context (Eq. 9)
        uint32_t vw[8];
        {
          const uint32_t cw[4] = {vc.x, vc.y, vc.z, vc.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int left = keep - 4 * j;
            const uint32_t w = cw[j] & (left >= 4 ? 0xFFFFFFFFu : (left <= 0 ? 0u : (1u << (8 * left)) - 1u));
            vw[2 * j] = p.kv_e5m2 ? e5m2x2_to_f16x2_lo(w) : e4m3x2_to_f16x2_lo(w);
            vw[2 * j + 1] = p.kv_e5m2 ? e5m2x2_to_f16x2_hi(w) : e4m3x2_to_f16x2_hi(w);
          }
        }
        *reinterpret_cast<uint4*>(vrow + (2 * c) * 128) = make_uint4(vw[0], vw[1], vw[2], vw[3]);
        *reinterpret_cast<uint4*>(vrow + (2 * c + 1) * 128) = make_uint4(vw[4], vw[5], vw[6], vw[7]);
        tmem_ld_wait(s);
        uint32_t pw[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float x0 = ex2(__uint_as_float(s[2 * e]) * sk - m_use), x1 = ex2(__uint_as_float(s[2 * e + 1]) * sk - m_use);
          const float p0 = (2 * e <= visible) ? x0 : 0.0f, p1 = (2 * e + 1 <= visible) ? x1 : 0.0f;
          l_row += p0 + p1;
          pw[e] = pack_f16x2(p0 * pv, p1 * pv);           // at most 256: probabilities are carried times 2^8
        }
        *reinterpret_cast<uint4*>(prow + (2 * c) * 128) = make_uint4(pw[0], pw[1], pw[2], pw[3]);
        *reinterpret_cast<uint4*>(prow + (2 * c + 1) * 128) = make_uint4(pw[4], pw[5], pw[6], pw[7]);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) { mbar_arrive(&bar_sfree[buf]); mbar_arrive(&bar_vread[vq]); }
      fence_proxy_async();
      mbar_arrive(&bar_pfull[team]);
    }

    // ---- the last P V instruction has finished: normalise and store ---------------------------------------
    if (!bad) {
      // A wait names a phase by its parity, which only tells the phase before from the one in progress: a team
      // that is done a tile early must not ask for the last tile's phase while the phase before it on the same
      // barrier is still open.  The last two tiles' instructions are waited for in order (the one before them
      // is finished: the team waited for it, or for a later one, inside its loop).
      const int tl = n_tiles - 1;
      bool ok = true;
      if (tl >= 1) ok = wait_bar(&bar_vdone[(tl - 1) % kPuVSlots], static_cast<uint32_t>((tl - 1) / kPuVSlots) & 1u, abort_flag);
      ok = ok && wait_bar(&bar_vdone[tl % kPuVSlots], static_cast<uint32_t>(tl / kPuVSlots) & 1u, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      bad = !ok;
    }
    xch[4 * kPuRows + part * kPuRows + r] = l_row;
    bad = barrier_or(1, kPuSm, bad);
    if (!bad) {
      tc_fence_after();
      const float l_all = (xch[4 * kPuRows + r] + xch[5 * kPuRows + r]) + (xch[6 * kPuRows + r] + xch[7 * kPuRows + r]);
      const float k = l_all > 0.0f ? v_max / (kPuGain * l_all) : 0.0f;
      // the four threads of row r store 32 dims each
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t o[16];
        tmem_ld16_issue(tmem_o + part * 32 + 16 * c + lane_base, o);
        tmem_ld_wait(o);
        if (live) {
          uint32_t w[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) w[j] = pack_bf16x2(__uint_as_float(o[2 * j]) * k, __uint_as_float(o[2 * j + 1]) * k);
          uint4* dst = reinterpret_cast<uint4*>(p.out + grow * D + part * 32 + 16 * c);
          dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
          dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
        }
      }
      tc_fence_before();
    }
    if (bad && r == 0) atomicCAS(p.status, 0, COOPT_ERR_TIMEOUT);
  }

  // ---- exit: copies still in flight get a bounded time to land, tensor memory is returned -----------
  __syncthreads();
  if (*abort_flag != 0 && warp == kPuProducer && lane == 0) {
    for (int slot = 0; slot < kPuSlots; ++slot)
      if ((pend_mask >> slot) & 1u) mbar_wait_bounded(&bar_full[slot], (pend_par >> slot) & 1u);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kPuSWarp) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512) : "memory");
}

}  // namespace

int launch_paged_prefill_umma(const coopt_cache* c, const void* q, void* out, const int32_t* cu_q_lens, const int32_t* block_table,
                              int32_t max_blocks_per_seq, const int32_t* context_lens, int32_t batch, int32_t num_q_heads,
                              int32_t total_q, int32_t causal, float sm_scale, void* workspace, cudaStream_t stream) {
  PrefillUmmaParams p;
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
  p.tile_queries = 128 / p.group;
  p.causal = causal;
  p.kv_e5m2 = c->dtype == COOPT_KV_FP8_E5M2 ? 1 : 0;
  p.sm_scale_log2 = sm_scale * kPuLog2e;
  p.status = static_cast<int*>(workspace);
  const long long tiles = static_cast<long long>(total_q) / p.tile_queries + batch;   // every sequence adds at most one partly filled tile
  if (tiles > 0x7fffffffll) return COOPT_ERR_UNSUPPORTED;
  CUtensorMap map_part, map_hdr;
  const long long granules = static_cast<long long>(c->num_blocks) * c->num_kv_heads;
  if (!encode_cache_map(&map_part, c->data, granules, PuCfg::kGran, PuCfg::kPart / 8) ||
      !encode_cache_map(&map_hdr, c->data, granules, PuCfg::kGran, kFp8Header / 8))
    return COOPT_ERR_CUDA;
  if (!configure_kernel_smem(reinterpret_cast<const void*>(&paged_prefill_umma_kernel), PuCfg::kSmemBytes)) return COOPT_ERR_CUDA;
  const dim3 grid(static_cast<unsigned>(tiles), static_cast<unsigned>(c->num_kv_heads));
  paged_prefill_umma_kernel<<<grid, kPuThreads, PuCfg::kSmemBytes, stream>>>(p, map_part, map_hdr);
  return cudaGetLastError() == cudaSuccess ? COOPT_OK : COOPT_ERR_CUDA;
}

}  // namespace coopt
