// Chunked prefill against the paged FP8 cache on the 5th-generation tensor cores (head_dim 128): Eq. 1
// with the causal K_{<=t}, Eq. 6 dequantisation on load, Eq. 7-8 grouped-query sharing, Eq. 9 valid
// blocks only, Eq. 10 max-subtracted softmax, for runs of several query tokens per sequence.
//
// A CTA owns one (sequence, kv head, tile of consecutive query tokens).  Its 128 rows are the (query
// token, query head of the group) pairs of the tile, so the K/V stream of the kv head is fetched once
// for all G heads (Algorithm 2).
//     S [128 rows x 128 keys] = Q  [128 x D] . Ktile^T      kind::f8f6f4: the cache codes as they are, Q as two E4M3
//                                                            terms of the bf16 query, both operands in shared memory
//     O [128 rows x D]       += P  [128 x 128 keys] . Vtile  kind::f16: P rounded once to f16 and read from tensor
//                                                            memory, the V codes widened to f16 (exact) in shared memory
// with fp32 accumulators in tensor memory.  The K scale of a block multiplies the logits of its 16 keys,
// the V scale is folded into the probabilities.  (Carrying P as E4M3 terms instead, three per probability for
// the same 11 bits, kept the V codes as they are but cost five conversions per pair of probabilities on the
// SM's conversion pipe; widening V costs a few integer instructions per pair of codes, and a tile of V is a
// sixteenth of a tile of P per query row.)
//
// The context is walked once, 128 keys (eight cache blocks) at a time; even tiles go to softmax team 0, odd
// tiles to team 1, and each team keeps an online softmax of its own for all 128 rows: a reference maximum per
// row, the sum of the exponentials taken against it, and an output accumulator of its own in tensor memory.
// The reference is lazy: a probability may exceed one by up to 2^8 before its row's reference is moved up to
// the row's maximum (and a V scale may exceed the team's reference scale by up to 2^4), because moving a
// reference means reading, scaling and writing back the row's 128 accumulators; f16 probabilities have room
// for that factor, and after the first tiles a reference hardly ever moves.  At the end the two teams'
// results are merged like two split-KV pieces.  Per tile the tensor core does 8 instructions for the logits
// and 8 for P V; nothing is computed twice.
//
// Tensor memory (512 columns): the logits of team b's tile in columns 128 b .. 128 b + 127, its accumulator in
// 256 + 128 b ...  A team writes its probabilities, two f16 to a column, over logits it has already consumed
// (keys 0-63 of the tile in columns 0-31 of its buffer, keys 64-127 in columns 64-95), so a team's next logits
// can be computed only once the P V instructions of its tile before are done; the other team's tile and the
// widening of the next V tile fill that time.
//
// Warp roles (608 threads):
//   warps 0-7, 8-15  two softmax teams.  Two threads of a team share row r: warps 0-3 of the team take the
//               tile's first four cache blocks, warps 4-7 the last four, in both passes over the logits (a first
//               pass for the maximum, a second for the probabilities); the two halves' maxima meet through
//               shared memory.  Before a tile's logits arrive, the team widens the tile's V^T into one of its two
//               f16 operands (the other may still be read by the P V instructions of the tile before);
//   warp 16     copies: gather requests over the tensor map of the cache into two slots for K tiles, freed as
//               soon as the logits are computed, and two slots for V tiles with the tile's scales, freed as
//               soon as the team has widened the codes;
//   warp 17     one lane issues the S instructions; warp 18 one lane issues the P V instructions.
// Every wait is bounded; a wait that runs out is reported in the status word and all roles leave through
// the common exit, which frees the tensor memory.
#include "coopt_trace.cuh"
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
constexpr int kPuSlots = 4;                                // of the copy ring: slots 0-1 take K tiles, slots 2-3 V tiles and scales
constexpr float kPuLog2e = 1.4426950408889634f;
constexpr float kPuMaxLag = 8.0f;                          // a row's reference may lag its maximum by this much (base-2 logarithm units)
constexpr float kPuScaleLag = 16.0f;                       // a V scale may exceed the team's reference scale by this factor

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
  unsigned long long* trace;   // trace build only: per CTA the cycles team 0's first thread spent in each phase
};

struct PuCfg {
  static constexpr int kPart = kBlockSize * kPuD;                 // 2048: K (or V) codes of one granule
  static constexpr int kGran = granule_bytes(kPuD, true);
  static constexpr int kKArea = kPuTileBlocks * kPart;            // 16 KB: the K parts, or the V parts, of a tile
  static constexpr int kHdrOff = kKArea;                          // V slots: behind the parts the eight headers (scales) of the tile
  static constexpr int kKSlot = kKArea;
  static constexpr int kVSlot = kKArea + kPuTileBlocks * kFp8Header;   // 16,640
  static constexpr int kOperand = 128 * 128;                      // one 128 x 128 operand of codes
  static constexpr int kOperand16 = 128 * 128 * 2;                // one 128 x 128 operand of f16 values
  static constexpr int kRingOff = 0;                              // K slot 0, K slot 1, V slot 0, V slot 1
  static constexpr int kVRingOff = kRingOff + 2 * kKSlot;
  static constexpr int kQOff = kVRingOff + 2 * kVSlot;            // Q: lead term, remainder term
  static constexpr int kV16Off = kQOff + 2 * kOperand;            // V^T of a tile widened to f16: [team][parity of the team's tile]
  static constexpr int kBarOff = kV16Off + 4 * kOperand16;
  static constexpr int kNumBars = kPuSlots + 2 + 2 + 2 + 2 + 2;   // full, kdone, vdone, vread, sfull, pfull
  static constexpr int kMiscOff = kBarOff + kNumBars * 8;
  static constexpr int kXchOff = kMiscOff + 64;                   // [team][parity][half][row] upper halves of fp32 maxima
  static constexpr int kSclOff = kXchOff + 2 * 2 * 2 * kPuRows * 2;   // [team][block][K scale, V scale] of the tile being worked on
  static constexpr int kSmemBytes = kSclOff + 2 * kPuTileBlocks * 2 * 4;
  static_assert(kVSlot % 128 == 0 && kQOff % 128 == 0 && kSmemBytes <= 232448, "shared memory of one CTA");
};

// 16 consecutive fp32 columns of this thread's tensor-memory lane, written back.
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
               ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
                 "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]) : "memory");
}
// Two E4M3 codes (bytes of `w` picked by `sel`: 0x1404 the low two, 0x3424 the high two) as two f16 holding the
// codes' values divided by 2^8, exactly: with the code in the upper byte of a half, its exponent and mantissa
// bits are moved down one place into the f16 fields (bias 7 against 15; a subnormal code becomes a subnormal
// f16 of the same proportion), the sign stays.  Integer instructions only: the conversion instruction shares
// the unit that takes the exponentials.
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2_small(uint32_t w, uint32_t sel) {
  const uint32_t x = __byte_perm(w, 0u, sel);
  return ((x >> 1) & 0x3F803F80u) | (x & 0x80008000u);
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

template <bool kE5m2>
__global__ void __launch_bounds__(kPuThreads, 1) paged_prefill_umma_kernel(const PrefillUmmaParams p, const __grid_constant__ CUtensorMap map_part,
                                                                          const __grid_constant__ CUtensorMap map_hdr) {
  using C = PuCfg;
  constexpr int D = kPuD;
  extern __shared__ __align__(128) uint8_t smem[];
  uint8_t* kring = smem + C::kRingOff;
  uint8_t* vring = smem + C::kVRingOff;
  uint8_t* qbuf = smem + C::kQOff;
  uint8_t* v16buf = smem + C::kV16Off;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::kBarOff);
  uint64_t* bar_full = bars;                         // [4] the copies into the slot have landed (K slots 0-1, V slots 2-3)
  uint64_t* bar_kdone = bar_full + kPuSlots;         // [2] the logits of the K tile in the slot are computed
  uint64_t* bar_vdone = bar_kdone + 2;               // [2] the P V instructions of the team's tile are done
  uint64_t* bar_vread = bar_vdone + 2;               // [2] the team has widened the V tile in the slot (and read its scales)
  uint64_t* bar_sfull = bar_vread + 2;               // [2] logits of a tile are in tensor memory (buffer = tile & 1 = team)
  uint64_t* bar_pfull = bar_sfull + 2;               // [2] the team's probabilities of a tile are in tensor memory, its V operand in shared memory
  unsigned short* xch = reinterpret_cast<unsigned short*>(smem + C::kXchOff);
  int* misc = reinterpret_cast<int*>(smem + C::kMiscOff);   // [0] sequence, [1] first query, [2] abort flag, [3] tensor memory
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
    for (int i = 0; i < kPuSlots; ++i) mbar_init(&bar_full[i], 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bar_kdone[i], 1); mbar_init(&bar_vdone[i], 1); mbar_init(&bar_vread[i], 8);
      mbar_init(&bar_sfull[i], 1); mbar_init(&bar_pfull[i], kPuTeam);
    }
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
  // index of the last visible key of the row.  Rows past the tile's last query (their query operand is zero and
  // they are never stored) see everything, so that their warp takes the same unmasked path as its live rows.
  const int lim = live ? (p.causal ? min(L - 1, L - n_new + q0 + qi) : L - 1) : (1 << 30);

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
  const uint32_t tmem_o = tmem + 256;                 // logits buffer b at column 128 b, team b's output at 256 + 128 b
  const uint32_t lane_base = static_cast<uint32_t>(warp & 3) * 32u << 16;
  uint32_t pend_mask = 0, pend_par = 0;               // copy lane: the latest phase expected of every slot it has filled

  if (warp == kPuProducer) {
    // ================= copies: the K parts of tile t into K slot t % 2, its V parts and headers into V slot t % 2 ====
    // Lane 3 q + w (q = 0, 1; w = 0, 1, 2) fetches the K parts (w = 0), the V parts (w = 1) or the headers
    // (w = 2) of granules 4 q .. 4 q + 3 of the tile.  Rows past the last block repeat the tile's first one.
    bool ok = true;
    const int q4 = lane / 3, what = lane - 3 * q4;
    const int x = what * (C::kPart / 8);
    const uint32_t dst_off = what == 2 ? C::kHdrOff + q4 * 4 * kFp8Header : q4 * 4 * C::kPart;       // inside the slot
    const CUtensorMap* map = what == 2 ? &map_hdr : &map_part;
    // The physical blocks are looked up 32 at a time (four tiles, one per lane), a batch ahead of their use, so
    // that the copy lane never waits for the block table (range-checked: a bad id is reported in the status
    // word and replaced by block 0, never dereferenced).
    const int* trow = p.block_table + static_cast<size_t>(b) * p.max_blocks_per_seq;
    const int nbatch = (n_tiles + 3) / 4;
    auto load_batch = [&](int lb) -> int {
      if (lb >= nbatch) return 0;
      const int j = lb * 32 + lane;
      int id = j < n_blocks ? trow[j] : 0;
      if (id < 0 || id >= p.num_blocks) { atomicCAS(p.status, 0, COOPT_ERR_INVALID_ARG); id = 0; }
      return id;
    };
    int cur_lb = 0;
    int ids_cur = load_batch(0), ids_next = load_batch(1);
    for (int t = 0; t < n_tiles; ++t) {
      const int nb = min(kPuTileBlocks, n_blocks - t * kPuTileBlocks);
      const int ngroups = (nb + 3) / 4;
      const int lb = t >> 2;
      if (lb != cur_lb) { ids_cur = ids_next; cur_lb = lb; ids_next = load_batch(lb + 1); }
      int rows[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int j = (q4 & 1) * 4 + i;                             // block of the tile (lanes past the six copy lanes fetch along)
        rows[i] = __shfl_sync(0xffffffffu, ids_cur, (t & 3) * 8 + (j < nb ? j : 0)) * Hkv + g;
      }
      const int sl = t & 1;
      const uint32_t use = static_cast<uint32_t>(t >> 1);
      // The V parts and the scales are requested as soon as the team has widened the V tile that was in the slot
      // (early in its work on that tile), the K parts once the logits of the K tile in the slot exist.  (The
      // slots' users before are the team's tile two back; a wait for phase k follows the one for phase k - 1.)
      if (lane == 0) {
        if (t >= 2) ok = wait_bar(&bar_vread[sl], (use - 1) & 1u, abort_flag);
        if (ok) {
          mbar_expect_tx(&bar_full[2 + sl], ngroups * 4 * (C::kPart + kFp8Header));
          pend_mask |= 4u << sl;
          pend_par = (pend_par & ~(4u << sl)) | ((use & 1u) << (2 + sl));
        }
      }
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      if (lane < 3 * ngroups && what != 0) gather4_g2s(vring + sl * C::kVSlot + dst_off, map, x, rows[0], rows[1], rows[2], rows[3], &bar_full[2 + sl]);
      if (lane == 0) {
        if (t >= 2) ok = wait_bar(&bar_kdone[sl], (use - 1) & 1u, abort_flag);
        if (ok) {
          mbar_expect_tx(&bar_full[sl], ngroups * 4 * C::kPart);
          pend_mask |= 1u << sl;
          pend_par = (pend_par & ~(1u << sl)) | ((use & 1u) << sl);
        }
      }
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      if (lane < 3 * ngroups && what == 0) gather4_g2s(kring + sl * C::kKSlot + dst_off, map, x, rows[0], rows[1], rows[2], rows[3], &bar_full[sl]);
    }
    if (!ok && lane == 0) atomicCAS(p.status, 0, COOPT_ERR_TIMEOUT);
  } else if (warp == kPuSWarp) {
    // ================= logits: S = Q . Ktile^T, both terms of Q (one lane) ====================================
    if (lane == 0) {
      bool ok = true;
      const uint64_t desc_k = umma_desc(smem_u32(kring), 128, 8 * D), desc_q = umma_desc(smem_u32(qbuf), 128, 1024);
      for (int t = 0; t < n_tiles && ok; ++t) {
        const uint32_t buf = t & 1u, use = static_cast<uint32_t>(t >> 1);
#ifdef COOPT_TRACE
        const long long ts0 = clock64();
#endif
        ok = wait_bar(&bar_full[buf], use & 1u, abort_flag);
#ifdef COOPT_TRACE
        const long long ts1 = clock64();
#endif
        // the buffer also holds the probabilities of the team's tile before, until their P V instructions are done
        if (ok && use > 0) ok = wait_bar(&bar_vdone[buf], (use - 1) & 1u, abort_flag);
        if (!ok) break;
#ifdef COOPT_TRACE
        if (p.trace != nullptr && blockIdx.y * gridDim.x + blockIdx.x < kTraceMaxCtas) {
          unsigned long long* out = p.trace + static_cast<size_t>(blockIdx.y * gridDim.x + blockIdx.x) * kTraceSlots;
          out[8] += ts1 - ts0; out[9] += clock64() - ts1;
        }
#endif
        tc_fence_after();
        const uint64_t dk = desc_k + ((buf * C::kKSlot) >> 4);
#pragma unroll
        for (int term = 0; term < 2; ++term)
#pragma unroll
          for (int ks = 0; ks < D / 32; ++ks)
            umma_f8(tmem + 128 * buf, desc_q + ((term * C::kOperand) >> 4) + ks * 16, dk + ks * 16, umma_idesc(128, 0, kE5m2 ? 1 : 0), (term | ks) != 0);
        umma_commit(&bar_sfull[buf]);
      }
      if (!ok) atomicCAS(p.status, 0, COOPT_ERR_TIMEOUT);
    }
  } else if (warp == kPuPvWarp) {
    // ================= outputs: O_team += P . Vtile (one lane) ===============================================
    if (lane == 0) {
      bool ok = true;
      // P is read from tensor memory, where the team left it over its own logits (keys 0-63 of the tile in columns
      // 0-31 of the team's buffer, keys 64-127 in columns 64-95); V^T is f16 in shared memory, K-major: 8 rows x 16
      // bytes (8 values) per core matrix, cores of a row group 128 bytes apart along the keys, row groups 2048 bytes apart
      const uint64_t desc_v = umma_desc(smem_u32(v16buf), 128, 2048);
      for (int t = 0; t < n_tiles && ok; ++t) {
        const uint32_t team = t & 1u, use = static_cast<uint32_t>(t >> 1);
#ifdef COOPT_TRACE
        const long long tp0 = clock64();
#endif
        ok = wait_bar(&bar_pfull[team], use & 1u, abort_flag);
        if (!ok) break;
#ifdef COOPT_TRACE
        if (p.trace != nullptr && blockIdx.y * gridDim.x + blockIdx.x < kTraceMaxCtas)
          p.trace[static_cast<size_t>(blockIdx.y * gridDim.x + blockIdx.x) * kTraceSlots + 10] += clock64() - tp0;
        const long long tp1 = clock64();
#endif
        tc_fence_after();
        const int nb = min(kPuTileBlocks, n_blocks - t * kPuTileBlocks);      // 16 keys (one cache block) per instruction
        const uint64_t dv = desc_v + (((team * 2 + (use & 1u)) * C::kOperand16) >> 4);
        const uint32_t p_cols = tmem + 128 * team;
        if (nb == kPuTileBlocks) {                        // all but a context's last tile: eight instructions in a row
#pragma unroll
          for (int ks = 0; ks < kPuTileBlocks; ++ks)
            umma_f16_ts(tmem_o + 128 * team, p_cols + (ks < 4 ? 8 * ks : 64 + 8 * (ks - 4)), dv + ks * 16, umma_idesc(D), (use | ks) != 0);
        } else {
          for (int ks = 0; ks < nb; ++ks)
            umma_f16_ts(tmem_o + 128 * team, p_cols + (ks < 4 ? 8 * ks : 64 + 8 * (ks - 4)), dv + ks * 16, umma_idesc(D), (use | ks) != 0);
        }
        umma_commit(&bar_vdone[team]);      // the team's logits buffer and this V operand are free again, its accumulator is at rest
#ifdef COOPT_TRACE
        {
          const long long ti = clock64();
          wait_bar(&bar_vdone[team], use & 1u, abort_flag);          // (measuring only: how long the instructions take to finish)
          if (p.trace != nullptr && blockIdx.y * gridDim.x + blockIdx.x < kTraceMaxCtas) {
            unsigned long long* out = p.trace + static_cast<size_t>(blockIdx.y * gridDim.x + blockIdx.x) * kTraceSlots;
            out[11] += ti - tp1; out[12] += clock64() - ti;
          }
        }
#endif
      }
      if (!ok) atomicCAS(p.status, 0, COOPT_ERR_TIMEOUT);
    }
  } else {
    // ================= softmax teams ================================================================================
    const int team = warp >> 3;
    const int tt = tid & (kPuTeam - 1);           // this thread within its team
    const int c_lo = half * (kPuTileBlocks / 2);  // the first of this thread's four cache blocks of a tile
    bool bad = false;
    float m_ref = -INFINITY;     // the row's reference maximum (the same in both threads of the row)
    float l_row = 0.0f;          // this thread's share of the row's sum of exponentials, against m_ref
    float v_ref = 0.0f;          // the team's reference V scale (uniform over the team)
    const uint32_t o_cols = tmem_o + 128 * team + 64 * half + lane_base;               // this thread's 64 of the row's accumulators
    const uint8_t* st = vring + team * C::kVSlot;                                      // the team's V slot: V parts, then the scales
    const uint32_t s_cols = tmem + 128 * team + lane_base;                             // the team's logits buffer
    float* scl = reinterpret_cast<float*>(smem + C::kSclOff) + team * (2 * kPuTileBlocks);   // the tile's [block][K scale, V scale]

    // A wait that runs out is made known to the whole team by the named barrier behind it, and the team leaves
    // the loop together; the other roles give up on their own waits once the abort flag is up.
#ifdef COOPT_TRACE
    long long tr_wait_in = 0, tr_pass_a = 0, tr_wait_pv = 0, tr_widen = 0, tr_pass_b = 0, tr_skew = 0, tr_t = clock64();
    const long long tr_start = tr_t;
#define PF_TRACE(acc) do { const long long now_ = clock64(); acc += now_ - tr_t; tr_t = now_; } while (0)
#else
#define PF_TRACE(acc) do { } while (0)
#endif
    // The loops over a tile are kept rolled (32 logits = two cache blocks per trip to tensor memory): unrolled,
    // the body of this loop was tens of KB of instructions and the teams waited for instruction fetch.
    for (int t = team; t < n_tiles && !bad; t += 2) {
      const uint32_t use = static_cast<uint32_t>(t >> 1);
      const int key0 = t * kPuTileKeys;
      const int nkeys = min(kPuTileKeys, kv_end - key0);
      const int nb = (nkeys + kBlockSize - 1) / kBlockSize;
      const int nb_mine = min(nb - c_lo, kPuTileBlocks / 2);                 // this thread's blocks of the tile (<= 0: none)
      // ---- the tile's V parts and scales have landed: V^T widened into one of the team's two f16 operands ---------
      // (the one that the P V instructions of the team's tile before do not read; those of the tile before that were
      // done before this tile's logits could be started).  One warp of the team watches the barrier; the other
      // seven wait for it on a named barrier, where the hardware parks them, instead of polling along with it.
      if ((warp & 7) == 0) {
        const bool ok = wait_bar(&bar_full[2 + team], use & 1u, abort_flag);
        bad = !__all_sync(0xffffffffu, ok);
      }
      bad = barrier_or(1 + team, kPuTeam, bad);           // uniform over the team from here
      if (bad) break;
      PF_TRACE(tr_wait_in);
      // the scales move to a place of the team's own: both passes need them after the V slot has been handed back
      if (tt < 2 * kPuTileBlocks) scl[tt] = reinterpret_cast<const float*>(st + C::kHdrOff)[(tt >> 1) * 8 + (tt & 1)];
      uint8_t* vrow = v16buf + (team * 2 + (use & 1u)) * C::kOperand16 + (r >> 3) * 2048 + (r & 7) * 16;    // dim r of V^T
#pragma unroll 1
      for (int ci = 0; ci < nb_mine; ++ci) {
        const int c = c_lo + ci;
        // dim r of V^T, the 16 tokens of block c: widened to f16 (exact; E4M3 codes come out divided by 2^8)
        const uint4 vc = *reinterpret_cast<const uint4*>(st + c * C::kPart + (r >> 3) * 128 + (r & 7) * 16);
        const int keep = nkeys - c * kBlockSize;          // tokens of the block inside the context (Eq. 9)
        uint32_t cw[4] = {vc.x, vc.y, vc.z, vc.w}, vw[8];
        if (keep < kBlockSize) {                          // the context ends inside this block: codes past it are cleared
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int left = keep - 4 * j;
            cw[j] &= left >= 4 ? 0xFFFFFFFFu : (left <= 0 ? 0u : (1u << (8 * left)) - 1u);
          }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          vw[2 * j] = kE5m2 ? e5m2x2_to_f16x2_lo(cw[j]) : e4m3x2_to_f16x2_small(cw[j], 0x1404u);
          vw[2 * j + 1] = kE5m2 ? e5m2x2_to_f16x2_hi(cw[j]) : e4m3x2_to_f16x2_small(cw[j], 0x3424u);
        }
        *reinterpret_cast<uint4*>(vrow + (2 * c) * 128) = make_uint4(vw[0], vw[1], vw[2], vw[3]);
        *reinterpret_cast<uint4*>(vrow + (2 * c + 1) * 128) = make_uint4(vw[4], vw[5], vw[6], vw[7]);
      }
      fence_proxy_async();                                // the tensor core will read what this thread has just written
      __syncwarp();
      if (lane == 0) mbar_arrive(&bar_vread[team]);       // the V slot may take the team's next tile
      PF_TRACE(tr_widen);

      // ---- the tile's logits ------------------------------------------------------------------------------------
      if ((warp & 7) == 0) {
        const bool ok = wait_bar(&bar_sfull[team], use & 1u, abort_flag);
        // the logits are computed: the tile's K slot can be refilled
        if (ok && lane == 0) mbar_arrive(&bar_kdone[team]);
        bad = !__all_sync(0xffffffffu, ok);
      }
      bad = barrier_or(1 + team, kPuTeam, bad);
      if (bad) break;
      tc_fence_after();
      PF_TRACE(tr_wait_pv);

      // ---- first pass: the maximum of this thread's half of the row; the tile's largest V scale ------------------
      float m_half = -INFINITY, v_tile = 0.0f;
#pragma unroll
      for (int c = 0; c < kPuTileBlocks; ++c) v_tile = fmaxf(v_tile, c < nb ? scl[2 * c + 1] : 0.0f);
#pragma unroll 1
      for (int ci = 0; ci < nb_mine; ci += 2) {
        const int c = c_lo + ci;
        uint32_t s[32];
        tmem_ld32_issue(s_cols + 16 * c, s);
        const bool two = ci + 1 < nb_mine;
        const float sk_a = scl[2 * c] * qscale, sk_b = two ? scl[2 * c + 2] * qscale : 0.0f;
        // keys 0 .. visible of the two blocks are seen by the row (Eq. 1: K_{<=t}; Eq. 9: none past the context)
        const int visible = min(lim - (key0 + c * kBlockSize), two ? 2 * kBlockSize - 1 : kBlockSize - 1);
        tmem_ld_wait32(s);
        if (visible < 2 * kBlockSize - 1) {
#pragma unroll
          for (int j = 0; j < 32; ++j) s[j] = j <= visible ? s[j] : 0xFF800000u;      // -inf
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          float mx[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) mx[j] = __uint_as_float(s[16 * h + j]);
#pragma unroll
          for (int j = 4; j < 16; ++j) mx[j & 3] = fmaxf(mx[j & 3], __uint_as_float(s[16 * h + j]));
          // a K scale is not negative, so a block's largest logit is its largest accumulator times the scale
          const float m_blk = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
          if (m_blk > -INFINITY) m_half = fmaxf(m_half, m_blk * (h ? sk_b : sk_a));
        }
      }
      // The two threads of a row tell each other their half's maximum, cut to its upper 16 bits, and both take the
      // larger of the two cut values as the tile's: a reference need not be the exact maximum, but the two must
      // agree on it.
      unsigned short* xrow = xch + (team * 2) * kPuRows + r;
      xrow[half * kPuRows] = static_cast<unsigned short>(__float_as_uint(m_half) >> 16);
      bad = barrier_or(1 + team, kPuTeam, bad);
      if (bad) break;
      PF_TRACE(tr_pass_a);
      const float m_tile = fmaxf(__uint_as_float(static_cast<uint32_t>(xrow[0]) << 16), __uint_as_float(static_cast<uint32_t>(xrow[kPuRows]) << 16));
      // lazy references: moved only when the tile would push a probability (or a scale ratio) past the margin
      const bool move_m = m_tile > m_ref + kPuMaxLag;             // also true for the row's first visible key (m_ref = -inf)
      const bool move_v = v_tile > v_ref * kPuScaleLag;           // uniform over the team; true for the first non-zero scale
      const float m_new = move_m ? m_tile : m_ref;
      const float v_new = move_v ? v_tile : v_ref;
      // the factor that brings what has been accumulated so far onto the new references
      float factor = 1.0f;
      if (move_m) factor = m_ref == -INFINITY ? 0.0f : ex2(m_ref - m_new);
      if (move_v) factor *= v_ref > 0.0f ? __fdividef(v_ref, v_new) : 0.0f;
      // Tensor-memory accesses are warp-wide: the warp rescales if any of its rows has to (the others by 1).  The
      // accumulator is at rest: the P V instructions of the team's tile before were done before this tile's logits
      // were started.
      const bool rescale = __any_sync(0xffffffffu, move_m || move_v) && use > 0;
      if (rescale) {
#pragma unroll 1
        for (int i = 0; i < 4; ++i) {
          uint32_t o[16];
          tmem_ld16_issue(o_cols + 16 * i, o);
          tmem_ld_wait(o);
#pragma unroll
          for (int j = 0; j < 16; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * factor);
          tmem_st16(o_cols + 16 * i, o);
        }
      }
      if (move_m) l_row *= m_ref == -INFINITY ? 0.0f : ex2(m_ref - m_new);
      m_ref = m_new;
      v_ref = v_new;
      const float m_use = m_ref == -INFINITY ? 0.0f : m_ref;
      const float v_inv = v_ref > 0.0f ? 1.0f / v_ref : 0.0f;

      // ---- second pass: probabilities of this thread's blocks against the reference (f16) ----------------------
      // p * pv = 2^(s * sk - m + log2 pv): the V scale rides in the exponent, and a block's sum of p is recovered
      // from the sum of p * pv with one division.  A V scale of zero (an all-zero block: its codes are zero too)
      // is replaced by a tiny one, a K scale of zero likewise (so that a masked logit stays -inf).  The
      // probabilities of 32 keys, two to a column, go back to tensor memory over the first half of the 32 logits
      // this thread has consumed most recently: the tensor core takes P from there.
#pragma unroll 1
      for (int ci = 0; ci < nb_mine; ci += 2) {
        const int c = c_lo + ci;
        uint32_t s[32];
        tmem_ld32_issue(s_cols + 16 * c, s);
        const bool two = ci + 1 < nb_mine;
        const float sk_a = fmaxf(scl[2 * c] * qscale, 1e-30f), sk_b = fmaxf(two ? scl[2 * c + 2] * qscale : 0.0f, 1e-30f);
        const float pv_a = fmaxf(scl[2 * c + 1] * v_inv, 0x1p-24f), pv_b = fmaxf(two ? scl[2 * c + 3] * v_inv : 0.0f, 0x1p-24f);   // at most 2^4
        const int visible = min(lim - (key0 + c * kBlockSize), two ? 2 * kBlockSize - 1 : kBlockSize - 1);
        tmem_ld_wait32(s);
        if (visible < 2 * kBlockSize - 1) {
#pragma unroll
          for (int j = 0; j < 32; ++j) s[j] = j <= visible ? s[j] : 0xFF800000u;
        }
        uint32_t pw[16];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const float sk = h ? sk_b : sk_a, pv = h ? pv_b : pv_a;
          float lg;
          asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(lg) : "f"(pv));
          const float shift = lg - m_use;
          float l_a = 0.0f, l_b = 0.0f;
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const float y0 = ex2(fmaf(__uint_as_float(s[16 * h + 2 * e]), sk, shift)), y1 = ex2(fmaf(__uint_as_float(s[16 * h + 2 * e + 1]), sk, shift));
            l_a += y0;
            l_b += y1;
            pw[8 * h + e] = pack_f16x2(y0, y1);           // at most 2^8 * 2^4: well inside f16
          }
          l_row += __fdividef(l_a + l_b, pv);
        }
        tmem_st16(s_cols + 64 * half + 8 * ci, pw);       // keys 16 c .. 16 c + 31 of the tile
      }
      tmem_st_wait();                                      // the probabilities (and a rescaled accumulator) are in place
      tc_fence_before();
      mbar_arrive(&bar_pfull[team]);
      PF_TRACE(tr_pass_b);
#ifdef COOPT_TRACE
      if (tid == 0) { wait_bar(&bar_pfull[team], use & 1u, abort_flag); PF_TRACE(tr_skew); }   // (measuring only: until the team's last thread has arrived)
#endif
    }
#ifdef COOPT_TRACE
    if (tid == 0 && p.trace != nullptr) {
      const int rec = blockIdx.y * gridDim.x + blockIdx.x;
      if (rec < kTraceMaxCtas) {
        unsigned long long* out = p.trace + static_cast<size_t>(rec) * kTraceSlots;
        out[0] = n_tiles; out[1] = tr_wait_in; out[2] = tr_pass_a; out[3] = tr_wait_pv; out[4] = tr_pass_b; out[5] = clock64() - tr_start; out[7] = tr_widen; out[13] = tr_skew;
      }
    }
#endif

    // ---- the team's last P V instruction has finished: the two teams' results are merged and stored ------------
    const int my_tiles = n_tiles > team ? (n_tiles - team + 1) / 2 : 0;
    if (!bad && my_tiles > 0 && (warp & 7) == 0) {
      bool ok = wait_bar(&bar_vdone[team], static_cast<uint32_t>(my_tiles - 1) & 1u, abort_flag);
      bad = !__all_sync(0xffffffffu, ok);
    }
    bad = barrier_or(1 + team, kPuTeam, bad);
    // what the other team needs of this one, in this team's own (now idle) V operand: per row its reference and
    // the two halves' sums, and the team's reference scale
    float* mine = reinterpret_cast<float*>(v16buf + team * 2 * C::kOperand16);
    const float* theirs = reinterpret_cast<const float*>(v16buf + (team ^ 1) * 2 * C::kOperand16);
    mine[half * kPuRows + r] = l_row;
    if (half == 0) mine[2 * kPuRows + r] = m_ref;
    if (tid == team * kPuTeam) mine[3 * kPuRows] = v_ref;
    bad = barrier_or(3, kPuSm, bad);
    if (!bad) {
      tc_fence_after();
      const float l_me = mine[r] + mine[kPuRows + r], l_ot = theirs[r] + theirs[kPuRows + r];
      const float m_ot = theirs[2 * kPuRows + r], v_ot = theirs[3 * kPuRows];
      const float M = fmaxf(l_me > 0.0f ? m_ref : -INFINITY, l_ot > 0.0f ? m_ot : -INFINITY);
      const float w_me = l_me > 0.0f ? ex2(m_ref - M) : 0.0f, w_ot = l_ot > 0.0f ? ex2(m_ot - M) : 0.0f;
      const float den = w_me * l_me + w_ot * l_ot;
      const float inv = den > 0.0f ? 1.0f / den : 0.0f;
      const float unit = kE5m2 ? 1.0f : 256.0f;        // the widened E4M3 codes carry their values / 2^8
      const float k_me = w_me * v_ref * inv * unit, k_ot = w_ot * v_ot * inv * unit;
      const bool other_ran = n_tiles > (team ^ 1);
      // the four threads of row r store 32 dims each
      const int part = team * 2 + half;
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t oa[16], ob[16];
        tmem_ld16_issue(tmem_o + 128 * team + part * 32 + 16 * c + lane_base, oa);
        tmem_ld_wait(oa);
        if (other_ran) {                                   // uniform; an accumulator that was never written holds anything
          tmem_ld16_issue(tmem_o + 128 * (team ^ 1) + part * 32 + 16 * c + lane_base, ob);
          tmem_ld_wait(ob);
        }
        if (live) {
          uint32_t w[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            float y0 = my_tiles > 0 && w_me > 0.0f ? __uint_as_float(oa[2 * j]) * k_me : 0.0f;
            float y1 = my_tiles > 0 && w_me > 0.0f ? __uint_as_float(oa[2 * j + 1]) * k_me : 0.0f;
            if (other_ran && w_ot > 0.0f) { y0 += __uint_as_float(ob[2 * j]) * k_ot; y1 += __uint_as_float(ob[2 * j + 1]) * k_ot; }
            w[j] = pack_bf16x2(y0, y1);
          }
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
  p.trace = nullptr;
#ifdef COOPT_TRACE
  p.trace = trace_buffer();
#endif
  const long long tiles = static_cast<long long>(total_q) / p.tile_queries + batch;   // every sequence adds at most one partly filled tile
  if (tiles > 0x7fffffffll) return COOPT_ERR_UNSUPPORTED;
  CUtensorMap map_part, map_hdr;
  const long long granules = static_cast<long long>(c->num_blocks) * c->num_kv_heads;
  if (!encode_cache_map(&map_part, c->data, granules, PuCfg::kGran, PuCfg::kPart / 8) ||
      !encode_cache_map(&map_hdr, c->data, granules, PuCfg::kGran, kFp8Header / 8))
    return COOPT_ERR_CUDA;
  const bool e5m2 = c->dtype == COOPT_KV_FP8_E5M2;
  const void* kernel = e5m2 ? reinterpret_cast<const void*>(&paged_prefill_umma_kernel<true>) : reinterpret_cast<const void*>(&paged_prefill_umma_kernel<false>);
  if (!configure_kernel_smem(kernel, PuCfg::kSmemBytes)) return COOPT_ERR_CUDA;
  const dim3 grid(static_cast<unsigned>(tiles), static_cast<unsigned>(c->num_kv_heads));
  if (e5m2) paged_prefill_umma_kernel<true><<<grid, kPuThreads, PuCfg::kSmemBytes, stream>>>(p, map_part, map_hdr);
  else paged_prefill_umma_kernel<false><<<grid, kPuThreads, PuCfg::kSmemBytes, stream>>>(p, map_part, map_hdr);
  return cudaGetLastError() == cudaSuccess ? COOPT_OK : COOPT_ERR_CUDA;
}

}  // namespace coopt
