// coopt_decode_plan: the work decomposition of a decode step, computed once and reused by every launch
// that shares the step's context lengths and block table (every layer of a model: Section 2's decode loop
// visits the same sequences, at the same lengths, once per layer).  Eq. 9: only the valid blocks of every
// sequence are listed.  CTA i of the kernel below works out what CTA i of the attention kernel will do --
// its slice of the flat (sequence, kv head, block) list, cut into segments and rounds, with the physical
// block ids already looked up and range-checked -- and leaves it in the plan buffer.
#include "coopt_plan.cuh"

namespace coopt {

namespace {

constexpr int kPlanThreads = 256;

struct PlanKernelParams {
  DecodeParams d;          // batch, heads, block table, context lengths, chunking, planned_ctas, status = plan status
  PlanHeader* header;
  uint8_t* regions;        // CTA regions of the plan
  int cta_stride;
  int key;
};

__global__ void __launch_bounds__(kPlanThreads) decode_plan_kernel(const PlanKernelParams pk) {
  __shared__ int pre_blk[kMaxBatch + 4];
  __shared__ int pre_unit[kMaxBatch + 4];
  __shared__ __align__(16) Segment segs[kMaxSeg];
  __shared__ __align__(16) int ids[kCap];
  __shared__ int misc[8];
  __shared__ long long slice[8];
  __shared__ int round_status;     // what the round being planned wants reported (bad block ids)
  __shared__ long long bounds[kMaxAnchorCtas + 1];
  __shared__ int budget[kMaxAnchorCtas];
  DecodeParams p = pk.d;
  p.status = &round_status;
  if (threadIdx.x == 0) round_status = 0;
  PlanSmem plan;
  plan.pre_blk = pre_blk; plan.pre_unit = pre_unit; plan.segs = segs; plan.ids = ids; plan.misc = misc; plan.slice = slice;
  plan.bounds = bounds;
  const int tid = threadIdx.x;
  int ctx_early[2];
  plan_prefix_load(p, tid, kPlanThreads, ctx_early);
  plan_prefix(p, plan, tid, kPlanThreads, ctx_early);
  if (!plan_anchor_bounds(p, plan, tid, kPlanThreads, budget)) plan.bounds = nullptr;
  if (tid == 0) plan_slice_publish(p, plan);
  __syncthreads();
  PlanSlice sl;
  const bool active = plan_slice_fetch(plan, sl);
  if (blockIdx.x == 0) {
    PlanHeader* h = pk.header;
    if (tid == 0) {
      h->magic = kPlanMagic; h->planned_ctas = p.planned_ctas; h->batch = p.batch; h->num_kv_heads = p.num_kv_heads;
      h->chunk_blocks = p.chunk_blocks; h->max_blocks_per_seq = p.max_blocks_per_seq; h->cta_stride = pk.cta_stride;
      h->num_blocks = p.num_blocks; h->max_chunks = p.max_chunks; h->status = 0;
    }
    for (int w = tid; w < kMaxBatch / 32; w += kPlanThreads) {
      unsigned int bits = 0;
      for (int i = 0; i < 32; ++i) {
        const int b = w * 32 + i;
        if (b < p.batch && pre_blk[b + 1] == pre_blk[b]) bits |= 1u << i;
      }
      h->empty_bits[w] = bits;
    }
  }

  uint8_t* region = pk.regions + static_cast<size_t>(blockIdx.x) * pk.cta_stride;
  int at = 0;                                   // bytes of the region used so far
  long long x = active ? sl.lo : 0;
  const long long x_end = active ? sl.hi : 0;
  bool wrote_last = false;
  // the anchor (anchored split): a whole (sequence, kv head) appended behind the CTA's last round of the remainder
  const int anchor_blocks = (active && sl.anchor_b >= 0) ? pre_blk[sl.anchor_b + 1] - pre_blk[sl.anchor_b] : 0;
  bool anchor_pending = anchor_blocks > 0;
  while (x < x_end || anchor_pending) {
    if (tid == 0) {
      if (x < x_end) {
        plan_round(p, plan, sl, x);
      } else {
        misc[0] = 0;
        misc[1] = static_cast<int>(x & 0xffffffffll);
        misc[2] = static_cast<int>(x >> 32);
      }
    }
    __syncthreads();
    int nseg = misc[0];
    const long long x_next = (static_cast<long long>(misc[2]) << 32) | static_cast<unsigned int>(misc[1]);
    if (tid < nseg) plan_round_finish(p, plan, sl, tid);
    __syncthreads();
    if (anchor_pending && x_next >= x_end) {
      int staged = 0;
      for (int i = 0; i < nseg; ++i) staged = max(staged, segs[i].list_off + segs[i].n);
      if (nseg < kMaxSeg && staged + anchor_blocks <= kCap) {      // else: a round of its own, next time round
        if (tid == 0) {
          Segment sg = {};
          sg.b = sl.anchor_b; sg.g = sl.anchor_g; sg.j0 = 0; sg.n = anchor_blocks; sg.list_off = staged;
          sg.partial = 0; sg.expected = 1; sg.seq_blocks = anchor_blocks;
          sg.run_flags = kRunFirst | kRunLast | kRunWhole | kSegTail;
          sg.run_expected = 1; sg.first_cta = static_cast<int>(blockIdx.x);
          segs[nseg] = sg;
        }
        ++nseg;
        anchor_pending = false;
      }
    }
    __syncthreads();
    plan_stage_ids(p, plan, nseg, tid, kPlanThreads);
    __syncthreads();
    int used = 0, n_tail = 0;
    for (int i = 0; i < nseg; ++i) { used = max(used, segs[i].list_off + segs[i].n); n_tail += (segs[i].run_flags & kSegTail) ? 1 : 0; }
    const int bytes = 64 + nseg * 64 + ((used * 4 + 15) / 16) * 16;
    if (at + bytes + 64 > pk.cta_stride) {       // cannot happen with the host's sizing; reported by the round written below
      if (tid == 0) round_status = COOPT_ERR_WORKSPACE;
      __syncthreads();
      break;
    }
    PlanRound* hdr = reinterpret_cast<PlanRound*>(region + at);
    if (tid == 0) {
      PlanRound h = {};
      h.nseg = nseg; h.n_ids = used; h.bytes = bytes; h.last = (x_next >= x_end && !anchor_pending) ? 1 : 0; h.n_tail = n_tail; h.key = pk.key;
      h.status = round_status;
      *hdr = h;
      round_status = 0;
    }
    int4* dseg = reinterpret_cast<int4*>(region + at + 64);
    const int4* sseg = reinterpret_cast<const int4*>(segs);
    for (int i = tid; i < nseg * 4; i += kPlanThreads) dseg[i] = sseg[i];
    int* dids = reinterpret_cast<int*>(region + at + 64 + nseg * 64);
    for (int i = tid; i < ((used + 3) / 4) * 4; i += kPlanThreads) dids[i] = i < used ? ids[i] : 0;
    wrote_last = x_next >= x_end && !anchor_pending;
    at += bytes;
    x = x_next;
    __syncthreads();
  }
  if (!wrote_last && tid == 0) {
    // a CTA without work (or whose plan did not fit): one empty, final round
    PlanRound h = {};
    h.nseg = 0; h.n_ids = 0; h.bytes = 64; h.last = 1; h.n_tail = 0; h.key = pk.key; h.status = round_status;
    *reinterpret_cast<PlanRound*>(region + (at + 64 <= pk.cta_stride ? at : 0)) = h;
  }
}

}  // namespace

// Bytes of one CTA region, from what the host knows: batch, kv heads, the width of the block table and the chunking.
int plan_cta_stride(int planned_ctas, int batch, int num_kv_heads, int max_blocks_per_seq, int chunk_blocks) {
  const long long n_max = static_cast<long long>(batch) * num_kv_heads * max_blocks_per_seq;
  long long blocks_max;
  if (chunk_blocks > 0) {
    const long long max_chunks = (max_blocks_per_seq + chunk_blocks - 1) / chunk_blocks;
    const long long u_max = static_cast<long long>(batch) * num_kv_heads * max_chunks;
    blocks_max = ((u_max + planned_ctas - 1) / planned_ctas + 1) * chunk_blocks;
  } else {
    blocks_max = (n_max + planned_ctas - 1) / planned_ctas + 1;
    // few blocks in all: fewer CTAs than planned take part, with at least kMinBlocksPerCta blocks each
    if (blocks_max < 2 * kMinBlocksPerCta) blocks_max = 2 * kMinBlocksPerCta;
  }
  blocks_max = blocks_max < n_max ? blocks_max : n_max;
  long long segs_max = blocks_max < static_cast<long long>(batch) * num_kv_heads ? blocks_max : static_cast<long long>(batch) * num_kv_heads;
  segs_max += 3;
  if (chunk_blocks > 0) segs_max += blocks_max / chunk_blocks + 1;
  if (segs_max > blocks_max + 2) segs_max = blocks_max + 2;
  const long long rounds_max = (segs_max + kMaxSeg - 1) / kMaxSeg + (blocks_max + kCap / 2 - 1) / (kCap / 2) + 1;
  const long long bytes = rounds_max * (64 + 16) + segs_max * 64 + blocks_max * 4 + 64;
  return static_cast<int>((bytes + 127) / 128 * 128);
}

size_t plan_bytes(int planned_ctas, int batch, int num_kv_heads, int max_blocks_per_seq, int chunk_blocks) {
  return kPlanHeaderBytes + static_cast<size_t>(planned_ctas) * plan_cta_stride(planned_ctas, batch, num_kv_heads, max_blocks_per_seq, chunk_blocks) +
         kPlanFirstChunk;      // a CTA's first fetch of a round may run past the end of the last region
}

int launch_decode_plan(const int32_t* block_table, int32_t max_blocks_per_seq, const int32_t* context_lens, int32_t batch,
                       int32_t num_kv_heads, int32_t num_blocks, int32_t chunk_size, int planned_ctas, void* plan,
                       cudaStream_t stream) {
  PlanKernelParams pk = {};
  DecodeParams& p = pk.d;
  p.block_table = block_table;
  p.context_lens = context_lens;
  p.max_blocks_per_seq = max_blocks_per_seq;
  p.batch = batch;
  p.num_kv_heads = num_kv_heads;
  p.num_blocks = num_blocks;
  p.planned_ctas = planned_ctas;
  p.chunk_blocks = chunk_size / kBlockSize;
  p.max_chunks = chunk_size > 0 ? static_cast<int>((static_cast<long long>(max_blocks_per_seq) * kBlockSize + chunk_size - 1) / chunk_size) : 0;
  pk.header = static_cast<PlanHeader*>(plan);
  pk.regions = static_cast<uint8_t*>(plan) + kPlanHeaderBytes;
  pk.cta_stride = plan_cta_stride(planned_ctas, batch, num_kv_heads, max_blocks_per_seq, p.chunk_blocks);
  pk.key = plan_key(planned_ctas, batch, num_kv_heads, p.chunk_blocks, max_blocks_per_seq, num_blocks);
  decode_plan_kernel<<<planned_ctas, kPlanThreads, 0, stream>>>(pk);
  return cudaGetLastError() == cudaSuccess ? COOPT_OK : COOPT_ERR_CUDA;
}

}  // namespace coopt
