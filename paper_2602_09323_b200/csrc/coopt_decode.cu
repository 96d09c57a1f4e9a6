// Paged decode over the bf16 ablation cache (the un-quantised layout the method is compared with):
// Eq. 1, Eq. 7-8 (the G query heads of a group consume one K/V stream), Eq. 9 (valid blocks only),
// Eq. 10 (max-subtracted softmax) and the Opt-Pa chunk-and-merge reduction, on mma.sync.  The FP8
// cache has its own kernel on the 5th-generation tensor cores; this file also holds the host launcher
// and the workspace arithmetic that both share.
//
// The work decomposition is the shared planner's.  Inside a segment the CTA's warps take blocks
// round-robin; each warp streams its granules through a private ring of shared-memory stages filled
// by bulk async copies (one elected lane issues, an mbarrier per stage counts the bytes), runs both
// contractions with the G query heads in the top rows of the 16-row instruction tile (the
// probabilities split into a bf16 high and low half, the low halves in rows 8..15), and keeps an
// online softmax per query head (warp shuffles inside the quad that owns a head, one shared-memory
// step across warps at the end of the segment).  A segment that does not cover its whole sequence
// leaves (m, l, o) in the workspace; the CTA that delivers the last piece of a (sequence, kv head)
// merges them by log-sum-exp and writes the bf16 output.
#include "coopt_plan.cuh"

namespace coopt {

namespace {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

template <int D>
struct Cfg {
  static constexpr int kGran = granule_bytes(D, false);
  static constexpr int kStages = 2;
  static constexpr int kKSteps = D / 16;
  static constexpr int kNTiles = D / 8;
  static constexpr int kOAcc = 4;               // accumulator registers kept per n-tile
  // shared memory carve-up (bytes)
  static constexpr int kRingOff = 0;
  static constexpr int kRingBytes = kWarps * kStages * kGran;
  static constexpr int kBarOff = kRingOff + kRingBytes;
  static constexpr int kIdsOff = kBarOff + kWarps * kStages * 8;
  static constexpr int kPreBlkOff = kIdsOff + kCap * 4;
  static constexpr int kPreUnitOff = kPreBlkOff + (kMaxBatch + 4) * 4;
  static constexpr int kSegOff = kPreUnitOff + (kMaxBatch + 4) * 4;
  static constexpr int kMergeOff = kSegOff + kMaxSeg * static_cast<int>(sizeof(Segment));
  static constexpr int kMergeStride = D + 4;    // floats per (warp, row): o[D], m, l, pad
  static constexpr int kMiscOff = kMergeOff + kWarps * kMaxGroup * kMergeStride * 4;
  static constexpr int kSmemBytes = kMiscOff + 128;
};

__device__ __forceinline__ float quad_max(float x) {
  x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 1));
  return fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 2));
}
__device__ __forceinline__ float quad_sum(float x) {
  x += __shfl_xor_sync(0xffffffffu, x, 1);
  return x + __shfl_xor_sync(0xffffffffu, x, 2);
}

// bf16 mma with only the top 8 rows of A in use (rows 8..15 are zero): two live accumulators.
__device__ __forceinline__ void mma_top(float& d0, float& d1, uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
  float t2, t3;
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%10,%10};"
               : "+f"(d0), "+f"(d1), "=f"(t2), "=f"(t3)
               : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1), "f"(0.0f));
  static_cast<void>(t2 + t3);
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1) paged_decode_kernel(const DecodeParams p) {
  using C = Cfg<D>;
  extern __shared__ __align__(128) uint8_t smem[];
  uint8_t* ring = smem + C::kRingOff;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::kBarOff);
  int* ids = reinterpret_cast<int*>(smem + C::kIdsOff);
  int* pre_blk = reinterpret_cast<int*>(smem + C::kPreBlkOff);
  int* pre_unit = reinterpret_cast<int*>(smem + C::kPreUnitOff);
  Segment* segs = reinterpret_cast<Segment*>(smem + C::kSegOff);
  float* merge = reinterpret_cast<float*>(smem + C::kMergeOff);
  int* misc = reinterpret_cast<int*>(smem + C::kMiscOff);   // [0] nseg, [1..2] next x, [3] last-arriver flag

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int row = lane >> 2, quad = lane & 3;
  const int B = p.batch, Hkv = p.num_kv_heads, G = p.group, Hq = p.num_q_heads;
  const bool chunk_mode = p.chunk_blocks > 0;

  // ---- plan: blocks (and chunks) per sequence, this CTA's slice of the flat block list ---------
  PlanSmem plan;
  plan.pre_blk = pre_blk; plan.pre_unit = pre_unit; plan.segs = segs; plan.ids = ids; plan.misc = misc;
  plan.slice = reinterpret_cast<long long*>(smem + C::kMiscOff + 64);
  plan.bounds = nullptr;
  int ctx_early[2];
  plan_prefix_load(p, tid, kThreads, ctx_early);
  if (tid == 0) {
    for (int i = 0; i < kWarps * C::kStages; ++i) mbar_init(&bars[i], 1);
    mbar_fence_init();
  }
  plan_prefix(p, plan, tid, kThreads, ctx_early);
  if (tid == 0) plan_slice_publish(p, plan);
  plan_check_single_query(p, tid, kThreads);
  __syncthreads();

  // sequences with an empty context: all-zero output rows
  for (int b = blockIdx.x; b < B; b += gridDim.x) {
    if (pre_blk[b + 1] == pre_blk[b])
      for (int i = tid; i < Hq * D; i += kThreads) p.out[static_cast<size_t>(b) * Hq * D + i] = __float2bfloat16(0.0f);
  }

  PlanSlice sl;
  if (!plan_slice_fetch(plan, sl)) return;
  const long long lo = sl.lo, hi = sl.hi;
  auto cta_of = [&](long long x) -> int { return plan_cta_of(sl, x); };

  // ---- per-warp pipeline state (persists across rounds) ----------------------------------------
  uint8_t* my_ring = ring + warp * C::kStages * C::kGran;
  uint64_t* my_bars = bars + warp * C::kStages;
  uint32_t issued = 0, consumed = 0;
  bool dead = false;   // a bounded wait ran out: stop touching the pipeline, keep the barriers' company

  long long x = lo;
  while (x < hi) {
    // ---- round: thread 0 plans up to kMaxSeg segments / kCap blocks starting at x -------------
    if (tid == 0) plan_round(p, plan, sl, x);
    __syncthreads();
    const int nseg = misc[0];
    const long long x_next = (static_cast<long long>(misc[2]) << 32) | static_cast<unsigned int>(misc[1]);
    if (tid < nseg) plan_round_finish(p, plan, sl, tid);
    plan_stage_ids(p, plan, nseg, tid, kThreads);
    __syncthreads();

    // ---- producer cursor of this warp: (segment, block-in-segment) --------------------------
    int pseg = 0, pk = warp;
    auto prod_normalise = [&]() {
      while (pseg < nseg && pk >= segs[pseg].n) { ++pseg; pk = warp; }
    };
    auto prod_issue = [&]() {
      const Segment& sg = segs[pseg];
      const int id = ids[sg.list_off + pk];
      const uint8_t* src = p.cache + (static_cast<size_t>(id) * Hkv + sg.g) * C::kGran;
      const uint32_t stage = issued % C::kStages;
      if (lane == 0) {
        mbar_expect_tx(&my_bars[stage], C::kGran);
        bulk_copy_g2s(my_ring + stage * C::kGran, src, C::kGran, &my_bars[stage]);
      }
      ++issued;
      pk += kWarps;
    };
    prod_normalise();
    if (!dead) {
#pragma unroll 1
      for (int s = 0; s < C::kStages && pseg < nseg; ++s) { prod_issue(); prod_normalise(); }
    }

    // raw query registers of the next segment, loaded one segment ahead
    uint32_t qraw[C::kKSteps][2];
    auto load_q_raw = [&](const Segment& sg) {
      const bool live = row < G;
      const __nv_bfloat16* qp = p.q + (static_cast<size_t>(sg.b) * Hq + sg.g * G + (live ? row : 0)) * D + 2 * quad;
#pragma unroll
      for (int s = 0; s < C::kKSteps; ++s) {
        qraw[s][0] = live ? *reinterpret_cast<const uint32_t*>(qp + 16 * s) : 0u;
        qraw[s][1] = live ? *reinterpret_cast<const uint32_t*>(qp + 16 * s + 8) : 0u;
      }
    };
    if (nseg > 0) load_q_raw(segs[0]);

    for (int si = 0; si < nseg; ++si) {
      const Segment sg = segs[si];

      // ---- query fragments (A operand): bf16 as loaded ---------------------------------------
      uint32_t qa[C::kKSteps][2];
#pragma unroll
      for (int s = 0; s < C::kKSteps; ++s) { qa[s][0] = qraw[s][0]; qa[s][1] = qraw[s][1]; }
      if (si + 1 < nseg) load_q_raw(segs[si + 1]);

      // ---- online softmax state of this warp for the segment ---------------------------------
      float m_run = -INFINITY, l_run = 0.0f;
      float o[C::kNTiles][C::kOAcc];
#pragma unroll
      for (int t = 0; t < C::kNTiles; ++t)
#pragma unroll
        for (int e = 0; e < C::kOAcc; ++e) o[t][e] = 0.0f;

#pragma unroll 1
      for (int k = warp; k < sg.n; k += kWarps) {
        const uint32_t stage = consumed % C::kStages;
        const uint32_t parity = (consumed / C::kStages) & 1u;
        if (!dead && !mbar_wait_bounded(&my_bars[stage], parity)) {
          dead = true;
          if (lane == 0) atomicCAS(p.status, 0, COOPT_ERR_TIMEOUT);
        }
        ++consumed;
        if (dead) continue;
        const uint8_t* st = my_ring + stage * C::kGran;
        const int nvalid = min(kBlockSize, sg.ctx_len - (sg.j0 + k) * kBlockSize);   // Eq. 9 tail

        // ---- S = Q K^T for 16 tokens (two n-tiles of 8) ---------------------------------------
        float s0[2] = {0.0f, 0.0f}, s1[2] = {0.0f, 0.0f};
        const uint8_t* kp = st + part_offset(D, false, 0) + lane * 16;
#pragma unroll
        for (int i = 0; i < D / 32; ++i) {
          const uint4 w0 = lds128(kp + (0 * (D / 32) + i) * 512);
          const uint4 w1 = lds128(kp + (1 * (D / 32) + i) * 512);
          mma_top(s0[0], s0[1], qa[2 * i][0], qa[2 * i][1], w0.x, w0.y);
          mma_top(s0[0], s0[1], qa[2 * i + 1][0], qa[2 * i + 1][1], w0.z, w0.w);
          mma_top(s1[0], s1[1], qa[2 * i][0], qa[2 * i][1], w1.x, w1.y);
          mma_top(s1[0], s1[1], qa[2 * i + 1][0], qa[2 * i + 1][1], w1.z, w1.w);
        }

        // ---- online softmax (Eq. 10), log2 units ---------------------------------------------------
        const float ks = p.sm_scale_log2;
        float sc[4] = {s0[0] * ks, s0[1] * ks, s1[0] * ks, s1[1] * ks};
        const int tok[4] = {2 * quad, 2 * quad + 1, 2 * quad + 8, 2 * quad + 9};
        if (nvalid < kBlockSize) {
#pragma unroll
          for (int e = 0; e < 4; ++e) sc[e] = tok[e] < nvalid ? sc[e] : -INFINITY;
        }
        const float m_blk = quad_max(fmaxf(fmaxf(sc[0], sc[1]), fmaxf(sc[2], sc[3])));
        const float m_new = fmaxf(m_run, m_blk);
        const float a_m = ex2(m_run - m_new);
        float pr[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) pr[e] = ex2(sc[e] - m_new);
        l_run = l_run * a_m + (pr[0] + pr[1]) + (pr[2] + pr[3]);
        m_run = m_new;
        if (__any_sync(0xffffffffu, a_m != 1.0f)) {
#pragma unroll
          for (int t = 0; t < C::kNTiles; ++t)
#pragma unroll
            for (int e = 0; e < C::kOAcc; ++e) o[t][e] *= a_m;
        }

        // ---- O += P V -----------------------------------------------------------------------------
        const uint8_t* vp = st + part_offset(D, false, 1) + lane * 16;
        {
          // bf16 probabilities split into high and low halves; the low halves ride in rows 8..15
          uint32_t hi0 = pack_bf16x2(pr[0], pr[1]), hi2 = pack_bf16x2(pr[2], pr[3]);
          const uint32_t lo0 = pack_bf16x2(pr[0] - bf16_lo(hi0), pr[1] - bf16_hi(hi0));
          const uint32_t lo2 = pack_bf16x2(pr[2] - bf16_lo(hi2), pr[3] - bf16_hi(hi2));
          uint32_t m01 = 0xffffffffu, m89 = 0xffffffffu;
          if (nvalid < kBlockSize) {
            m01 = (tok[0] < nvalid ? 0x0000FFFFu : 0u) | (tok[1] < nvalid ? 0xFFFF0000u : 0u);
            m89 = (tok[2] < nvalid ? 0x0000FFFFu : 0u) | (tok[3] < nvalid ? 0xFFFF0000u : 0u);
          }
#pragma unroll
          for (int qd = 0; qd < D / 16; ++qd) {
            const uint4 w = lds128(vp + qd * 512);
            mma16816<false>(o[2 * qd], hi0, lo0, hi2, lo2, w.x & m01, w.y & m89);
            mma16816<false>(o[2 * qd + 1], hi0, lo0, hi2, lo2, w.z & m01, w.w & m89);
          }
        }

        // ---- hand the stage back to the copy engine ------------------------------------------------
        __syncwarp();
        if (pseg < nseg) {
          if (lane == 0) fence_proxy_async();
          prod_issue();
          prod_normalise();
        }
      }

      // ---- end of segment: combine the warps' states through shared memory --------------------
      l_run = quad_sum(l_run);
      if (row < G) {
        float* mr = merge + (warp * kMaxGroup + row) * C::kMergeStride;
#pragma unroll
        for (int t = 0; t < C::kNTiles; ++t)   // high and low halves of the probabilities were accumulated apart
          *reinterpret_cast<float2*>(mr + 8 * t + 2 * quad) = make_float2(o[t][0] + o[t][2], o[t][1] + o[t][3]);
        if (quad == 0) { mr[D] = m_run; mr[D + 1] = l_run; }
      }
      __syncthreads();

      const int h0 = sg.g * G;
      float* po = nullptr; float* pm = nullptr; float* pl = nullptr;
      if (sg.partial) {
        if (chunk_mode) {
          const size_t base = (static_cast<size_t>(sg.b) * Hq + h0) * p.max_chunks + sg.slot;
          po = p.part_o + base * D; pm = p.part_m + base; pl = p.part_l + base;
        } else {
          const size_t base = static_cast<size_t>(sg.slot) * G;
          po = p.part_o + base * D; pm = p.part_m + base; pl = p.part_l + base;
        }
      }
      const size_t pstride = chunk_mode ? static_cast<size_t>(p.max_chunks) : 1;   // row stride of partial arrays
      for (int idx = tid; idx < G * D; idx += kThreads) {
        const int r = idx / D, d = idx % D;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) M = fmaxf(M, merge[(w * kMaxGroup + r) * C::kMergeStride + D]);
        float num = 0.0f, den = 0.0f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
          const float* mw = merge + (w * kMaxGroup + r) * C::kMergeStride;
          const float wgt = ex2(mw[D] - M);
          num += wgt * mw[d];
          den += wgt * mw[D + 1];
        }
        const float val = num / den;
        if (!sg.partial) {
          p.out[(static_cast<size_t>(sg.b) * Hq + h0 + r) * D + d] = __float2bfloat16(val);
        } else {
          po[r * pstride * D + d] = val;
          if (d == 0) {
            pm[r * pstride] = chunk_mode ? M * kLn2 : M;   // exported partials use natural-log units
            pl[r * pstride] = den;
          }
        }
      }

      if (sg.partial) {
        __threadfence();
        __syncthreads();
        int* counter = p.counters + sg.b * Hkv + sg.g;
        if (tid == 0) {
          const int old = atomicAdd(counter, 1);
          const int last = old == sg.expected - 1;
          if (last) *counter = 0;             // ready for the next call
          misc[3] = last;
        }
        __syncthreads();
        if (misc[3]) {
          // this CTA delivered the last piece: log-sum-exp merge of all pieces (split-K merge)
          __threadfence();
          int first_cta = 0;
          if (!chunk_mode) {
            const long long fs = static_cast<long long>(Hkv) * pre_blk[sg.b] + static_cast<long long>(sg.g) * sg.seq_blocks;
            first_cta = cta_of(fs);
          }
          for (int idx = tid; idx < G * D; idx += kThreads) {
            const int r = idx / D, d = idx % D;
            float M = -INFINITY;
            for (int c = 0; c < sg.expected; ++c) {
              size_t at;
              if (chunk_mode) at = (static_cast<size_t>(sg.b) * Hq + h0 + r) * p.max_chunks + c;
              else at = static_cast<size_t>(2 * (first_cta + c) + (c == 0 ? 1 : 0)) * G + r;
              M = fmaxf(M, __ldcg(p.part_m + at));
            }
            float num = 0.0f, den = 0.0f;
            for (int c = 0; c < sg.expected; ++c) {
              size_t at;
              if (chunk_mode) at = (static_cast<size_t>(sg.b) * Hq + h0 + r) * p.max_chunks + c;
              else at = static_cast<size_t>(2 * (first_cta + c) + (c == 0 ? 1 : 0)) * G + r;
              const float mc = __ldcg(p.part_m + at), lc = __ldcg(p.part_l + at);
              const float wgt = lc * (chunk_mode ? ex2((mc - M) * kLog2e) : ex2(mc - M));
              num += wgt * __ldcg(p.part_o + at * D + d);
              den += wgt;
            }
            p.out[(static_cast<size_t>(sg.b) * Hq + h0 + r) * D + d] = __float2bfloat16(num / den);
          }
        }
      }
      __syncthreads();   // merge scratch and misc[3] are reused by the next segment
    }

    x = x_next;
    __syncthreads();
  }

  // a warp that gave up still has copies in flight: give them a bounded time to land before
  // the CTA's shared memory is released
  if (dead) {
    while (consumed < issued) {
      const uint32_t stage = consumed % C::kStages, parity = (consumed / C::kStages) & 1u;
      mbar_wait_bounded(&my_bars[stage], parity);
      ++consumed;
    }
  }
}

}  // namespace

// Workspace layout: [header 256 B: word 0 = status][counters int32 x 16384][partials][plan of a one-off call].
size_t plan_bytes(int planned_ctas, int batch, int num_kv_heads, int max_blocks_per_seq, int chunk_blocks);
int plan_cta_stride(int planned_ctas, int batch, int num_kv_heads, int max_blocks_per_seq, int chunk_blocks);
int launch_decode_plan(const int32_t* block_table, int32_t max_blocks_per_seq, const int32_t* context_lens, int32_t batch,
                       int32_t num_kv_heads, int32_t num_blocks, int32_t chunk_size, int planned_ctas, void* plan,
                       cudaStream_t stream);

static size_t partials_bytes(int planned_ctas, int group, int head_dim, int batch, int num_q_heads, int max_chunks) {
  size_t bytes = kWsHeaderBytes + static_cast<size_t>(kCounterSlots) * 4;
  const size_t dec = static_cast<size_t>(2) * planned_ctas * group * (head_dim + 2) * 4;
  const size_t chk = static_cast<size_t>(batch) * num_q_heads * max_chunks * (head_dim + 2) * 4;
  // chunk mode holds both: the per-chunk partials it exports and the merged pieces of the CTAs' runs
  return (bytes + (max_chunks > 0 ? chk + dec + 256 : dec) + 256 + 255) / 256 * 256;
}
size_t decode_workspace_bytes(int planned_ctas, int group, int head_dim, int batch, int num_q_heads, int num_kv_heads,
                              int max_blocks_per_seq, int chunk_blocks, int max_chunks) {
  // calls that bring no plan of their own (coopt_paged_decode, coopt_paged_chunked) plan into the workspace
  return partials_bytes(planned_ctas, group, head_dim, batch, num_q_heads, max_chunks) +
         plan_bytes(planned_ctas, batch, num_kv_heads, max_blocks_per_seq, chunk_blocks);
}
size_t workspace_control_bytes() { return kWsHeaderBytes + static_cast<size_t>(kCounterSlots) * 4; }

int decode_planned_ctas(int num_sms, long long upper_blocks) {
  // a CTA's slice must fit one round of staged block ids, so that no (sequence, kv head) is cut twice
  // inside one CTA; slices differ by at most one block from the mean
  const long long need = (upper_blocks + (kCap - 16) - 1) / (kCap - 16);
  return static_cast<int>(need > num_sms ? need : num_sms);
}
int decode_max_batch() { return kMaxBatch; }
int decode_counter_slots() { return kCounterSlots; }
int decode_max_chunk_blocks() { return kCap; }

void chunk_partial_offsets(int batch, int num_q_heads, int head_dim, int max_chunks, size_t* o, size_t* m, size_t* l) {
  const size_t rows = static_cast<size_t>(batch) * num_q_heads * max_chunks;
  *o = workspace_control_bytes();
  *m = *o + rows * head_dim * 4;
  *l = *m + rows * 4;
}

template <int D>
static int launch_one(const DecodeParams& p, int grid, cudaStream_t stream) {
  using C = Cfg<D>;
  if (!configure_kernel_smem(reinterpret_cast<const void*>(&paged_decode_kernel<D>), C::kSmemBytes)) return COOPT_ERR_CUDA;
  paged_decode_kernel<D><<<grid, kThreads, C::kSmemBytes, stream>>>(p);
  return cudaGetLastError() == cudaSuccess ? COOPT_OK : COOPT_ERR_CUDA;
}

int launch_paged_decode_umma(const DecodeParams& p, int head_dim, int grid, bool overlap_previous, cudaStream_t stream);

// Everything of DecodeParams that does not depend on where the plan comes from.
static void fill_decode_params(DecodeParams& p, const coopt_cache* c, const void* q, void* out, const int32_t* block_table,
                               int32_t max_blocks_per_seq, const int32_t* context_lens, int32_t batch, int32_t num_q_heads,
                               float sm_scale, int32_t chunk_size, const int32_t* cu_q_lens, void* workspace, int planned_ctas) {
  p = DecodeParams{};
  p.cache = static_cast<const uint8_t*>(c->data);
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.out = static_cast<__nv_bfloat16*>(out);
  p.block_table = block_table;
  p.context_lens = context_lens;
  p.cu_q_lens = cu_q_lens;
  p.max_blocks_per_seq = max_blocks_per_seq;
  p.batch = batch;
  p.num_q_heads = num_q_heads;
  p.num_kv_heads = c->num_kv_heads;
  p.group = num_q_heads / c->num_kv_heads;
  p.num_blocks = c->num_blocks;
  p.kv_e5m2 = c->dtype == COOPT_KV_FP8_E5M2 ? 1 : 0;
  p.sm_scale_log2 = sm_scale * kLog2e;
  p.planned_ctas = planned_ctas;
  p.chunk_blocks = chunk_size / kBlockSize;
  p.max_chunks = chunk_size > 0 ? static_cast<int>((static_cast<long long>(max_blocks_per_seq) * kBlockSize + chunk_size - 1) / chunk_size) : 0;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  p.status = reinterpret_cast<int*>(ws);
  p.counters = reinterpret_cast<int*>(ws + kWsHeaderBytes);
  uint8_t* parts = ws + workspace_control_bytes();
  if (chunk_size > 0) {
    size_t o, m, l;
    chunk_partial_offsets(batch, num_q_heads, c->head_dim, p.max_chunks, &o, &m, &l);
    p.part_o = reinterpret_cast<float*>(ws + o);
    p.part_m = reinterpret_cast<float*>(ws + m);
    p.part_l = reinterpret_cast<float*>(ws + l);
    const size_t chunk_rows = static_cast<size_t>(batch) * num_q_heads * p.max_chunks;
    const size_t run_at = (l + chunk_rows * 4 + 255) / 256 * 256;
    const size_t rows = static_cast<size_t>(2) * planned_ctas * p.group;
    p.run_o = reinterpret_cast<float*>(ws + run_at);
    p.run_m = p.run_o + rows * c->head_dim;
    p.run_l = p.run_m + rows;
  } else {
    const size_t rows = static_cast<size_t>(2) * planned_ctas * p.group;
    p.part_o = reinterpret_cast<float*>(parts);
    p.part_m = p.part_o + rows * c->head_dim;
    p.part_l = p.part_m + rows;
    p.run_o = p.part_o;
    p.run_m = p.part_m;
    p.run_l = p.part_l;
  }
}

static void attach_plan(DecodeParams& p, const void* plan) {
  p.plan_header = static_cast<const PlanHeader*>(plan);
  p.plan = static_cast<const uint8_t*>(plan) + kPlanHeaderBytes;
  p.plan_cta_stride = plan_cta_stride(p.planned_ctas, p.batch, p.num_kv_heads, p.max_blocks_per_seq, p.chunk_blocks);
  p.plan_key = plan_key(p.planned_ctas, p.batch, p.num_kv_heads, p.chunk_blocks, p.max_blocks_per_seq, p.num_blocks);
}

// A call that brings no plan: the FP8 kernel's plan is made in the workspace first (one more small launch);
// the bf16 ablation kernel plans inside its own CTAs.
int launch_paged_decode(const coopt_cache* c, const void* q, void* out, const int32_t* block_table,
                        int32_t max_blocks_per_seq, const int32_t* context_lens, int32_t batch, int32_t num_q_heads,
                        float sm_scale, int32_t chunk_size, const int32_t* cu_q_lens, void* workspace, int planned_ctas,
                        cudaStream_t stream) {
  DecodeParams p;
  fill_decode_params(p, c, q, out, block_table, max_blocks_per_seq, context_lens, batch, num_q_heads, sm_scale, chunk_size,
                     cu_q_lens, workspace, planned_ctas);
  if (!is_fp8(c->dtype))
    return c->head_dim == 128 ? launch_one<128>(p, planned_ctas, stream) : launch_one<64>(p, planned_ctas, stream);
  void* plan = static_cast<uint8_t*>(workspace) + partials_bytes(planned_ctas, p.group, c->head_dim, batch, num_q_heads, p.max_chunks);
  const int rc = launch_decode_plan(block_table, max_blocks_per_seq, context_lens, batch, c->num_kv_heads, c->num_blocks, chunk_size,
                                    planned_ctas, plan, stream);
  if (rc != COOPT_OK) return rc;
  attach_plan(p, plan);
  return launch_paged_decode_umma(p, c->head_dim, planned_ctas, false, stream);
}

// A call that brings its plan (coopt_decode_plan) and may append one token per sequence in the same launch.
int launch_decode_planned(const coopt_cache* c, const void* plan, const void* k_new, const void* v_new, int64_t kv_token_stride,
                          const int64_t* slot_mapping, const void* q, void* out, int32_t max_blocks_per_seq, int32_t batch,
                          int32_t num_q_heads, float sm_scale, int32_t chunk_size, const int32_t* cu_q_lens, void* workspace,
                          int planned_ctas, bool overlap_previous, cudaStream_t stream) {
  DecodeParams p;
  fill_decode_params(p, c, q, out, nullptr, max_blocks_per_seq, nullptr, batch, num_q_heads, sm_scale, chunk_size, cu_q_lens,
                     workspace, planned_ctas);
  p.k_new = static_cast<const __nv_bfloat16*>(k_new);
  p.v_new = static_cast<const __nv_bfloat16*>(v_new);
  p.slot_mapping = reinterpret_cast<const long long*>(slot_mapping);
  p.kv_token_stride = kv_token_stride;
  attach_plan(p, plan);
  return launch_paged_decode_umma(p, c->head_dim, planned_ctas, overlap_previous, stream);
}

}  // namespace coopt
