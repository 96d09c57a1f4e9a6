// Work decomposition shared by the decode kernels (Eq. 9: only the valid blocks of every sequence
// are ever listed).  All (sequence, kv head, block) triples form one flat list.  In decode mode
// CTA i takes the i-th of P equal slices of the list (split-KV balanced by bytes); in chunk mode
// (Opt-Pa) it takes a contiguous run of fixed-size chunks.  A slice is cut into segments at
// (sequence, kv head) boundaries and at chunk boundaries; a CTA walks its slice in rounds of at
// most kMaxSeg segments / kCap blocks whose physical block ids are staged in shared memory.
#pragma once

#include "coopt_common.cuh"

namespace coopt {

constexpr int kCap = 2048;            // block ids staged in shared memory per round
constexpr int kMaxSeg = 32;           // segments planned per round
constexpr int kMaxBatch = 512;
constexpr int kMinBlocksPerCta = 16;
constexpr int kMaxGroup = 8;
constexpr int kCounterSlots = 16384;
constexpr int kWsHeaderBytes = 256;
constexpr int kMaxAnchorCtas = 256;   // the anchored split (below) is worked out for at most this many CTAs

struct Segment {
  int b, g;          // sequence, kv head
  int j0, n;         // first block of the sequence in this segment, number of blocks
  int list_off;      // position of block j0 in the staged id list
  int partial;       // 0: covers the whole sequence, write the output directly
  int slot;          // partial: workspace slot (decode mode) or chunk index (chunk mode)
  int expected;      // partial: number of pieces the (sequence, kv head) is cut into
  int seq_blocks;    // blocks of the whole sequence
  int ctx_len;       // tokens of the whole sequence
  // A run is what one CTA holds of one (sequence, kv head): in chunk mode several consecutive chunks,
  // which the tcgen05 kernel merges on chip before anything is counted; in decode mode the segment itself.
  int run_flags;     // kRunFirst | kRunLast | kRunWhole
  int run_slot;      // workspace slot of the run's merged piece (two per CTA)
  int run_expected;  // number of CTAs that hold a run of this (sequence, kv head)
  int first_cta;     // the first of them
  int pad[2];        // 64 bytes: segments are copied in 16-byte pieces
};
constexpr int kRunFirst = 1, kRunLast = 2, kRunWhole = 4;
constexpr int kSegTail = 8;    // the segment ends with the last block of its sequence (where a new token lands)

// A plan computed once (coopt_decode_plan) and read by every launch that shares its context lengths and
// block table: per planned CTA a region of `cta_stride` bytes holding its rounds back to back, each round a
// header, its segments and the staged physical block ids of those segments.
struct PlanHeader {          // first 256 bytes of a plan
  int magic, planned_ctas, batch, num_kv_heads;
  int chunk_blocks, max_blocks_per_seq, cta_stride, status;
  int num_blocks, max_chunks;
  unsigned int empty_bits[kMaxBatch / 32];   // bit b: sequence b has no context (its output rows are zeros)
  int pad[54 - kMaxBatch / 32];
};
struct PlanRound {           // 64 bytes in front of a round's segments
  int nseg;                  // 0: the CTA has nothing (left) to do
  int n_ids;
  int bytes;                 // of the whole round record (header, segments, ids), a multiple of 16
  int last;                  // 1: no round follows
  int n_tail;                // segments that carry kSegTail
  int key;                   // plan_key() of the problem the plan was made for
  int status;                // a coopt_status the planner wants reported (a block id out of range, a plan that did not fit)
  int pad[9];
};
// What a launch and the plan it is handed must agree on.
__host__ __device__ inline int plan_key(int planned_ctas, int batch, int num_kv_heads, int chunk_blocks, int max_blocks_per_seq, int num_blocks) {
  unsigned int h = 0x9e3779b9u;
  const int v[6] = {planned_ctas, batch, num_kv_heads, chunk_blocks, max_blocks_per_seq, num_blocks};
  for (int i = 0; i < 6; ++i) h = (h ^ static_cast<unsigned int>(v[i])) * 0x01000193u + 0x7f4a7c15u;
  return static_cast<int>(h | 1u);
}
constexpr int kPlanMagic = 0x434f5031;
constexpr int kPlanHeaderBytes = 256;
constexpr int kPlanFirstChunk = 4096;   // what a CTA fetches of a round before it knows the round's size
constexpr int kPlanRoundMax = 64 + kMaxSeg * 64 + kCap * 4;   // largest round record
static_assert(sizeof(PlanHeader) == kPlanHeaderBytes && sizeof(PlanRound) == 64 && sizeof(Segment) == 64, "plan layout");

struct DecodeParams {
  const uint8_t* cache;
  const __nv_bfloat16* q;
  __nv_bfloat16* out;
  const int* block_table;
  const int* context_lens;
  const int* cu_q_lens;    // chunk mode: prefix sums of the query tokens per sequence (must be 0..batch); else null
  const uint8_t* plan;     // FP8 kernel: the plan's CTA regions (behind the PlanHeader); cta_stride bytes each
  int plan_cta_stride;
  const PlanHeader* plan_header;
  int plan_key;            // what every round header of the plan must carry
  // fused append (all null / 0 when the call has no new tokens): Algorithm 1 phase 1 for one token per sequence
  const __nv_bfloat16* k_new;
  const __nv_bfloat16* v_new;
  const long long* slot_mapping;
  long long kv_token_stride;
  unsigned long long* trace;   // time stamps (trace build only; null otherwise)
  int plan_rotate;             // trace build only: CTA i works through plan region (i + plan_rotate) mod planned_ctas
  int max_blocks_per_seq;
  int batch, num_q_heads, num_kv_heads, group;
  int num_blocks;
  int kv_e5m2;             // 1: the cache codes are E5M2 (the format ablation), 0: E4M3
  float sm_scale_log2;     // sm_scale * log2(e)
  int planned_ctas;        // P
  int chunk_blocks;        // 0 = decode mode
  int max_chunks;
  int* status;
  int* counters;
  float* part_o;           // decode: [2P][G][D]        chunk: [B][Hq][max_chunks][D]
  float* part_m;           // decode: [2P][G]           chunk: [B][Hq][max_chunks]
  float* part_l;
  float* run_o;            // merged pieces of runs, [2P][G][D] (decode mode: the same arrays as part_*)
  float* run_m;            // [2P][G], base-2 logarithm units
  float* run_l;
};

#ifdef __CUDACC__

// Shared-memory arrays of the planner; the kernel owns the storage.
struct PlanSmem {
  int* pre_blk;      // [kMaxBatch + 4] prefix sums of blocks per sequence
  int* pre_unit;     // [kMaxBatch + 4] prefix sums of chunks per sequence (chunk mode)
  Segment* segs;     // [kMaxSeg]
  int* ids;          // [kCap]
  int* misc;         // [4]: nseg, next x (lo, hi), scratch flag
  long long* slice;  // [8]: the CTA's slice as one thread worked it out (plan_slice_publish)
  long long* bounds; // anchored split: [P + 1] first flat index of every CTA's slice of the remainder (nullptr: equal slices)
};

// floor(a / b) for 0 <= a < 2^52, 0 < b < 2^31: one double division and a fix-up instead of the
// generic 64-bit routine (the planner is one thread's serial work at the head of every CTA).
__device__ __forceinline__ long long plan_div(long long a, int b) {
  long long q = static_cast<long long>(static_cast<double>(a) / static_cast<double>(b));
  const long long r = a - q * b;
  if (r < 0) --q; else if (r >= b) ++q;
  return q;
}

__device__ __forceinline__ int plan_find_seq(const int* pre, int batch, long long x, int heads) {
  // largest b in [0, batch) with heads * pre[b] <= x
  int lo = 0, hi = batch - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (static_cast<long long>(heads) * pre[mid] <= x) lo = mid; else hi = mid - 1;
  }
  return lo;
}

// The context lengths this thread will turn into block counts: loaded as early as the kernel can, so
// that the trip to memory overlaps the rest of the set-up.  (kMaxBatch <= 2 * the smallest CTA.)
__device__ __forceinline__ void plan_prefix_load(const DecodeParams& p, int tid, int nthreads, int (&L)[2]) {
#pragma unroll
  for (int k = 0; k < 2; ++k) {
    const int b = tid + k * nthreads;
    L[k] = b < p.batch ? p.context_lens[b] : 0;
  }
}

// The decode kernels serve coopt_paged_chunked only when every sequence has exactly one query token.  The
// host sees no more than the total, so CTA 0 looks at the prefix sums themselves: any other split of the
// same total is reported in the status word (the rows are then attributed to the wrong sequences).
__device__ __forceinline__ void plan_check_single_query(const DecodeParams& p, int tid, int nthreads) {
  if (p.cu_q_lens == nullptr || blockIdx.x != 0) return;
  for (int b = tid; b <= p.batch; b += nthreads)
    if (p.cu_q_lens[b] != b) atomicCAS(p.status, 0, COOPT_ERR_INVALID_ARG);
}

// Blocks (and chunks) per sequence and their prefix sums.  Every thread of the CTA calls this.
__device__ inline void plan_prefix(const DecodeParams& p, const PlanSmem& s, int tid, int nthreads, const int (&Lin)[2]) {
  const int B = p.batch;
  const bool chunk_mode = p.chunk_blocks > 0;
#pragma unroll
  for (int k = 0; k < 2; ++k) {
    const int b = tid + k * nthreads;
    if (b >= B) break;
    int L = Lin[k];
    L = max(0, min(L, p.max_blocks_per_seq * kBlockSize));
    const int nb = (L + kBlockSize - 1) / kBlockSize;
    s.pre_blk[b + 1] = nb;
    s.pre_unit[b + 1] = chunk_mode ? (nb + p.chunk_blocks - 1) / p.chunk_blocks : 0;
  }
  if (tid == 0) { s.pre_blk[0] = 0; s.pre_unit[0] = 0; }
  __syncthreads();
  if (tid < 32) {
    const int lane = tid;
    int carry_b = 0, carry_u = 0;
    for (int base = 0; base < B; base += 32) {
      const int i = base + lane;
      int vb = i < B ? s.pre_blk[i + 1] : 0, vu = i < B ? s.pre_unit[i + 1] : 0;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int tb = __shfl_up_sync(0xffffffffu, vb, o), tu = __shfl_up_sync(0xffffffffu, vu, o);
        if (lane >= o) { vb += tb; vu += tu; }
      }
      if (i < B) { s.pre_blk[i + 1] = vb + carry_b; s.pre_unit[i + 1] = vu + carry_u; }
      carry_b += __shfl_sync(0xffffffffu, vb, 31);
      carry_u += __shfl_sync(0xffffffffu, vu, 31);
    }
  }
  __syncthreads();
}

// The slice [lo, hi) of the flat block list that belongs to this CTA; false if it has none.
struct PlanSlice {
  long long lo, hi, N;
  long long ulo, uhi, U;     // chunk mode: the same slice in units of (sequence, kv head, chunk)
  int P;
  const long long* bounds;   // anchored split: slice i of the remainder is [bounds[i], bounds[i + 1])
  int anchor_b, anchor_g;    // anchored split: the (sequence, kv head) this CTA also takes whole; -1: none
};
__device__ inline bool plan_slice(const DecodeParams& p, const PlanSmem& s, PlanSlice& sl) {
  const int B = p.batch, Hkv = p.num_kv_heads;
  sl.N = static_cast<long long>(Hkv) * s.pre_blk[B];
  sl.ulo = sl.uhi = sl.U = 0;
  sl.bounds = nullptr;
  sl.anchor_b = sl.anchor_g = -1;
  if (sl.N == 0) return false;
  if (p.chunk_blocks == 0) {
    sl.P = static_cast<int>(min(static_cast<long long>(p.planned_ctas), max(1ll, sl.N / kMinBlocksPerCta)));
    if (static_cast<int>(blockIdx.x) >= sl.P) return false;
    if (s.bounds != nullptr && sl.P == p.planned_ctas) {
      const int u = B * Hkv - sl.P + static_cast<int>(blockIdx.x);
      sl.bounds = s.bounds;
      sl.anchor_b = u / Hkv;
      sl.anchor_g = u - sl.anchor_b * Hkv;
      sl.lo = s.bounds[blockIdx.x];
      sl.hi = s.bounds[blockIdx.x + 1];
      return true;
    }
    sl.lo = plan_div(blockIdx.x * sl.N, sl.P);
    sl.hi = plan_div((blockIdx.x + 1ll) * sl.N, sl.P);
    return true;
  }
  const long long U = static_cast<long long>(Hkv) * s.pre_unit[B];
  sl.P = static_cast<int>(min(static_cast<long long>(p.planned_ctas), U));
  if (static_cast<int>(blockIdx.x) >= sl.P) return false;
  const long long ulo = plan_div(blockIdx.x * U, sl.P), uhi = plan_div((blockIdx.x + 1ll) * U, sl.P);
  auto unit_to_block = [&](long long u) -> long long {
    if (u >= U) return sl.N;
    const int b = plan_find_seq(s.pre_unit, B, u, Hkv);
    const int nch = s.pre_unit[b + 1] - s.pre_unit[b], nb = s.pre_blk[b + 1] - s.pre_blk[b];
    const long long rem = u - static_cast<long long>(Hkv) * s.pre_unit[b];
    const int g = static_cast<int>(plan_div(rem, nch)), c = static_cast<int>(rem - static_cast<long long>(g) * nch);
    return static_cast<long long>(Hkv) * s.pre_blk[b] + static_cast<long long>(g) * nb + static_cast<long long>(c) * p.chunk_blocks;
  };
  sl.lo = unit_to_block(ulo);
  sl.hi = unit_to_block(uhi);
  sl.ulo = ulo; sl.uhi = uhi; sl.U = U;
  return true;
}
// One thread works the slice out (its divisions are double-precision: a whole CTA doing them at once
// queues on the few units an SM has) and leaves it in shared memory; after a barrier everybody fetches it.
__device__ inline void plan_slice_publish(const DecodeParams& p, const PlanSmem& s) {
  PlanSlice sl;
  const bool active = plan_slice(p, s, sl);
  s.slice[0] = sl.lo; s.slice[1] = sl.hi; s.slice[2] = sl.N; s.slice[3] = sl.ulo; s.slice[4] = sl.uhi; s.slice[5] = sl.U;
  s.slice[6] = sl.P | (static_cast<long long>(sl.anchor_b + 1) << 32);
  s.slice[7] = (active ? 1 : 0) | (sl.bounds != nullptr ? 2 : 0) | (static_cast<long long>(sl.anchor_g + 1) << 32);
}
__device__ inline bool plan_slice_fetch(const PlanSmem& s, PlanSlice& sl) {
  sl.lo = s.slice[0]; sl.hi = s.slice[1]; sl.N = s.slice[2]; sl.ulo = s.slice[3]; sl.uhi = s.slice[4]; sl.U = s.slice[5];
  sl.P = static_cast<int>(s.slice[6] & 0xffffffffll);
  sl.anchor_b = static_cast<int>(s.slice[6] >> 32) - 1;
  sl.anchor_g = static_cast<int>(s.slice[7] >> 32) - 1;
  sl.bounds = (s.slice[7] & 2) ? s.bounds : nullptr;
  return (s.slice[7] & 1) != 0;
}
// CTA that owns flat block index x (decode mode).
__device__ __forceinline__ int plan_cta_of(const PlanSlice& sl, long long x) {
  if (sl.bounds != nullptr) {
    int lo = 0, hi = sl.P - 1;                       // largest i with bounds[i] <= x among the non-empty slices
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (sl.bounds[mid] <= x) lo = mid; else hi = mid - 1;
    }
    return lo;
  }
  return static_cast<int>(plan_div((x + 1) * sl.P - 1, static_cast<int>(sl.N)));
}

// Anchored split (decode mode).  With equal slices of the flat list, a CTA whose slice holds no whole
// (sequence, kv head) ends on a piece of a cut one, and is then usually the last to deliver a piece of it: the
// launch ends on its trip to the piece counter and its merge.  Here every CTA takes one (sequence, kv head)
// whole -- its anchor: the last P of them, in order -- and the others (the remainder, a prefix of the flat
// list) are cut so that every CTA still gets the same number of blocks: slice i of the remainder has the equal
// share minus the anchor's blocks.  A CTA works through its pieces of the remainder first and its anchor last,
// so every merge happens while the stream still runs and every CTA ends on a plain store.  Needs as many
// (sequence, kv head) pairs as CTAs and no anchor larger than the equal share; false otherwise.
__device__ inline bool plan_anchor_bounds(const DecodeParams& p, const PlanSmem& s, int tid, int nthreads, int* budget /* shared, [P] */) {
  const int B = p.batch, Hkv = p.num_kv_heads, P = p.planned_ctas;
  const long long N = static_cast<long long>(Hkv) * s.pre_blk[B];
  const long long U = static_cast<long long>(B) * Hkv;
  if (s.bounds == nullptr || p.chunk_blocks != 0 || P > kMaxAnchorCtas || U < P || N / kMinBlocksPerCta < P) return false;
  for (int i = tid; i < P; i += nthreads) {
    const int u = static_cast<int>(U) - P + i, b = u / Hkv;
    const int a = s.pre_blk[b + 1] - s.pre_blk[b];
    const long long share = plan_div((i + 1ll) * N, P) - plan_div(static_cast<long long>(i) * N, P);
    budget[i] = static_cast<int>(share) - a;
  }
  __syncthreads();
  if (tid == 0) {
    long long at = 0;
    bool ok = true, none = true, all = true;
    for (int i = 0; i < P; ++i) {
      s.bounds[i] = at;
      ok = ok && budget[i] >= 0;
      none = none && budget[i] == 0;
      all = all && budget[i] > 0;
      at += budget[i];
    }
    // the pieces of a cut (sequence, kv head) must sit in consecutive CTAs: no empty slice between two others
    s.bounds[P] = (ok && (none || all)) ? at : -1;
  }
  __syncthreads();
  return s.bounds[P] >= 0;
}

// One thread plans the next round starting at flat index x: fills the geometry of segs (plan_round_finish
// adds the rest), misc[0] = number of segments, misc[1..2] = where the following round starts.
__device__ inline void plan_round(const DecodeParams& p, const PlanSmem& s, const PlanSlice& sl, long long x) {
  const int B = p.batch, Hkv = p.num_kv_heads;
  const bool chunk_mode = p.chunk_blocks > 0;
  int nseg = 0, used = 0;
  long long xx = x;
  int cb = plan_find_seq(s.pre_blk, B, xx, Hkv), cg, cj;
  {
    const int nb = s.pre_blk[cb + 1] - s.pre_blk[cb];
    const long long rem = xx - static_cast<long long>(Hkv) * s.pre_blk[cb];
    cg = static_cast<int>(plan_div(rem, nb));
    cj = static_cast<int>(rem - static_cast<long long>(cg) * nb);
  }
  while (xx < sl.hi && nseg < kMaxSeg) {
    const int nb = s.pre_blk[cb + 1] - s.pre_blk[cb];
    long long n = min(static_cast<long long>(nb - cj), sl.hi - xx);
    if (chunk_mode) n = min(n, static_cast<long long>(p.chunk_blocks - cj % p.chunk_blocks));
    if (used + n > kCap) {
      if (nseg > 0) break;
      n = kCap;   // cannot happen with the host's sizing; keeps the kernel in bounds regardless
    }
    Segment sg;
    sg.b = cb; sg.g = cg; sg.j0 = cj; sg.n = static_cast<int>(n); sg.list_off = used;
    sg.seq_blocks = nb;
    sg.ctx_len = 0;     // filled in by plan_stage_ids, off this thread's serial path
    sg.partial = chunk_mode ? 1 : !(cj == 0 && n == nb);
    sg.slot = sg.expected = sg.run_flags = sg.run_slot = sg.run_expected = sg.first_cta = 0;   // plan_round_finish
    s.segs[nseg++] = sg;
    used += static_cast<int>(n);
    xx += n;
    cj += static_cast<int>(n);
    if (cj >= nb) {
      cj = 0;
      if (++cg == Hkv) {
        cg = 0;
        ++cb;
        while (cb < B && s.pre_blk[cb + 1] == s.pre_blk[cb]) ++cb;
      }
    }
  }
  // Decode mode: segments are independent, so the ones that cover their whole sequence go last.  A piece of
  // a cut sequence then reaches the workspace early, its merge (by whichever CTA delivers last) happens while
  // the stream still runs, and the CTA's own end is a plain store instead of a counter trip and a merge.
  // (Only the first and the last segment of a slice can be pieces of a cut sequence.)
  if (!chunk_mode && nseg > 1 && s.segs[nseg - 1].partial) {
    const int to = s.segs[0].partial ? 1 : 0;
    const Segment last = s.segs[nseg - 1];
    for (int i = nseg - 1; i > to; --i) s.segs[i] = s.segs[i - 1];
    s.segs[to] = last;
  }
  s.misc[0] = nseg;
  s.misc[1] = static_cast<int>(xx & 0xffffffffll);
  s.misc[2] = static_cast<int>(xx >> 32);
}

// What plan_round left out of segment k: the fields that cost divisions.  Thread k of the CTA calls this
// for k < number of segments, so the segments' divisions run side by side.
__device__ inline void plan_round_finish(const DecodeParams& p, const PlanSmem& s, const PlanSlice& sl, int k) {
  const int Hkv = p.num_kv_heads;
  const bool chunk_mode = p.chunk_blocks > 0;
  Segment& sg = s.segs[k];
  const int nb = sg.seq_blocks;
  {
    if (chunk_mode) {
      const int nch = s.pre_unit[sg.b + 1] - s.pre_unit[sg.b], c = sg.j0 / p.chunk_blocks;
      sg.slot = c;
      sg.expected = nch;
      // the CTA's run of this (sequence, kv head): units [max(fu, ulo), min(fu + nch, uhi))
      const long long fu = static_cast<long long>(Hkv) * s.pre_unit[sg.b] + static_cast<long long>(sg.g) * nch, u = fu + c;
      const int Un = static_cast<int>(sl.U);
      const int cta_f = static_cast<int>(plan_div((fu + 1) * sl.P - 1, Un)), cta_l = static_cast<int>(plan_div((fu + nch) * sl.P - 1, Un));
      sg.first_cta = cta_f;
      sg.run_expected = cta_l - cta_f + 1;
      sg.run_slot = 2 * blockIdx.x + (cta_f < static_cast<int>(blockIdx.x) ? 0 : 1);
      sg.run_flags = ((c == 0 || u == sl.ulo) ? kRunFirst : 0) | ((c == nch - 1 || u == sl.uhi - 1) ? kRunLast : 0) |
                     (cta_l == cta_f ? kRunWhole : 0) | (sg.j0 + sg.n == nb ? kSegTail : 0);
    } else {
      sg.slot = 2 * blockIdx.x + (sg.j0 > 0 ? 0 : 1);
      const long long fs = static_cast<long long>(Hkv) * s.pre_blk[sg.b] + static_cast<long long>(sg.g) * nb;
      sg.first_cta = plan_cta_of(sl, fs);
      sg.expected = plan_cta_of(sl, fs + nb - 1) - sg.first_cta + 1;
      sg.run_flags = kRunFirst | kRunLast | (sg.partial ? 0 : kRunWhole) | (sg.j0 + sg.n == nb ? kSegTail : 0);
      sg.run_slot = sg.slot;
      sg.run_expected = sg.expected;
    }
  }
}

// Physical block ids of every planned segment -> shared memory (range-checked: a bad id is
// reported in the status word and replaced by block 0, never dereferenced), and the context length
// of every segment's sequence.
__device__ inline void plan_stage_ids(const DecodeParams& p, const PlanSmem& s, int nseg, int tid, int nthreads) {
  if (tid < nseg) s.segs[tid].ctx_len = max(0, min(p.context_lens[s.segs[tid].b], p.max_blocks_per_seq * kBlockSize));
  for (int i = 0; i < nseg; ++i) {
    const Segment& sg = s.segs[i];
    const int* trow = p.block_table + static_cast<size_t>(sg.b) * p.max_blocks_per_seq + sg.j0;
    for (int k = tid; k < sg.n; k += nthreads) {
      int id = trow[k];
      if (id < 0 || id >= p.num_blocks) { atomicCAS(p.status, 0, COOPT_ERR_INVALID_ARG); id = 0; }
      s.ids[sg.list_off + k] = id;
    }
  }
}

#endif  // __CUDACC__

}  // namespace coopt
