// Shared device/host helpers of libcoopt: the cache layout, PTX wrappers, small utilities.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/coopt.h"

namespace coopt {

constexpr int kBlockSize = 16;     // tokens per physical block
constexpr int kFp8Header = 32;     // bytes behind the codes of an FP8 granule that are read: K scale, V scale, zeros
constexpr int kFp8Tail = 128;      // bytes behind the codes that the granule occupies: the header and padding, so that
                                   // granules start on 128-byte lines and no line is shared by two writers
constexpr float kE4m3Max = 448.0f;
constexpr float kE5m2Max = 57344.0f;
inline bool is_fp8(int dtype) { return dtype == COOPT_KV_FP8_E4M3 || dtype == COOPT_KV_FP8_E5M2; }

// ---- cache layout ---------------------------------------------------------------------------
// A granule holds 16 tokens x D of K and of V for one (block, kv head).
// FP8 granule: K part, V part, then the 32-byte header with the two scales (the V part and the header
// travel in one copy).  The parts have the layout the tensor cores read from shared memory without any
// rearrangement, so that a bulk copy is all the staging there is.  Both parts are "K-major, no swizzle"
// operands of tcgen05.mma: 8 rows x 16 bytes form a contiguous 128-byte core matrix.
//   K part (rows = tokens, contraction over dims): token t, dim d at
//       (t / 8) * 8D + (d / 16) * 128 + (t % 8) * 16 + d % 16
//   V part (rows = dims, contraction over tokens; i.e. V transposed): token t, dim d at
//       (d / 8) * 128 + (d % 8) * 16 + t
// bf16 granule (ablation cache, mma.sync kernel): values permuted so that lane `l` of a warp finds
// the B-operand registers of mma.m16n8k16 in consecutive 16-byte chunks:
//   K tile (QK^T: n = token, k = dim):   lane = 4 * (token % 8) + (dim % 8) / 2
//   V tile (P V : k = token, n = dim):   lane = 4 * (dim % 8)   + (token % 8) / 2
// a chunk holds two k-steps (K) or two n-tiles (V) of two registers each.

__host__ __device__ constexpr int granule_bytes(int D, bool fp8) {
  return fp8 ? kFp8Tail + 2 * kBlockSize * D : 2 * kBlockSize * D * 2;
}
__host__ __device__ constexpr int part_bytes(int D, bool fp8) { return kBlockSize * D * (fp8 ? 1 : 2); }
__host__ __device__ constexpr int part_offset(int D, bool fp8, int which) { return which * part_bytes(D, fp8); }
// FP8 granule: [K codes 16D][V codes 16D][fp32 K scale, fp32 V scale, 24 zero bytes][96 bytes of padding]
__host__ __device__ constexpr int header_offset(int D) { return 2 * kBlockSize * D; }

// Byte offset of K element (token t, dim d) inside the K part.
__host__ __device__ inline int k_elem_offset(int D, bool fp8, int t, int d) {
  if (fp8) return (t >> 3) * 8 * D + (d >> 4) * 128 + (t & 7) * 16 + (d & 15);
  const int nt = t >> 3, n = t & 7;
  const int s = d >> 4, r = d & 15;
  const int c = (r & 7) >> 1;
  const int lane = 4 * n + c;
  return ((nt * (D / 32) + (s >> 1)) * 32 + lane) * 16 + (s & 1) * 8 + (r >> 3) * 4 + (r & 1) * 2;
}

// Byte offset of V element (token t, dim d) inside the V part.
__host__ __device__ inline int v_elem_offset(int D, bool fp8, int t, int d) {
  if (fp8) return (d >> 3) * 128 + (d & 7) * 16 + t;
  const int n = d & 7;
  const int c = (t & 7) >> 1;
  const int lane = 4 * n + c;
  return ((d >> 4) * 32 + lane) * 16 + ((d & 15) >> 3) * 8 + (t >> 3) * 4 + (t & 1) * 2;
}

// ---- PTX wrappers -----------------------------------------------------------------------------
#ifdef __CUDACC__

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// Two E4M3 codes (low 16 bits of `w`, or high 16 bits) -> two f16 (exact).
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2_lo(uint32_t w) {
  uint32_t d;
  asm("{ .reg .b16 lo, hi; mov.b32 {lo, hi}, %1; cvt.rn.f16x2.e4m3x2 %0, lo; }" : "=r"(d) : "r"(w));
  return d;
}
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2_hi(uint32_t w) {
  uint32_t d;
  asm("{ .reg .b16 lo, hi; mov.b32 {lo, hi}, %1; cvt.rn.f16x2.e4m3x2 %0, hi; }" : "=r"(d) : "r"(w));
  return d;
}

// fp32 -> one E4M3 code, round to nearest even, saturating to +-448.
__device__ __forceinline__ uint32_t f32_to_e4m3(float x) {
  uint16_t d;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(d) : "f"(0.0f), "f"(x));
  return d & 0xFFu;
}

// fp32 -> one E5M2 code, round to nearest even, saturating to +-57344.
__device__ __forceinline__ uint32_t f32_to_e5m2(float x) {
  uint16_t d;
  asm("cvt.rn.satfinite.e5m2x2.f32 %0, %1, %2;" : "=h"(d) : "f"(0.0f), "f"(x));
  return d & 0xFFu;
}
// An E5M2 code is the upper byte of the half-precision number of the same value.
__device__ __forceinline__ float e5m2_to_f32(uint32_t code) {
  return __half2float(__ushort_as_half(static_cast<unsigned short>((code & 0xFFu) << 8)));
}
// Two E5M2 codes (bytes 0, 1 of `w`, or bytes 2, 3) -> two f16 (exact).
__device__ __forceinline__ uint32_t e5m2x2_to_f16x2_lo(uint32_t w) { return __byte_perm(w, 0u, 0x1404); }
__device__ __forceinline__ uint32_t e5m2x2_to_f16x2_hi(uint32_t w) { return __byte_perm(w, 0u, 0x3424); }

__device__ __forceinline__ float e4m3_to_f32(uint32_t code) {
  const uint32_t h2 = e4m3x2_to_f16x2_lo(code & 0xFFu);
  return __half2float(__ushort_as_half(static_cast<unsigned short>(h2 & 0xFFFFu)));
}

// D = A * B + C, 16x8x16, f16 inputs (FP8 cache) or bf16 inputs (bf16 cache), fp32 accumulate.
template <bool F16>
__device__ __forceinline__ void mma16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  if constexpr (F16) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
  } else {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
  }
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi) {
  const __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// ---- mbarrier + bulk copy (one elected lane issues; waits are bounded) -------------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Wait for a phase of the barrier; gives up after about kWaitLimitNs and returns false.
constexpr uint64_t kWaitLimitNs = 2000000000ull;
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_timer_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (global_timer_ns() - t0 > kWaitLimitNs) return false;
  }
}
// Untiled bulk copy global -> this CTA's shared memory; both addresses 16-byte aligned, bytes % 16 == 0.
__device__ __forceinline__ void bulk_copy_g2s(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst_smem)),
               "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ uint4 lds128(const void* p) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(smem_u32(p)));
  return v;
}

#endif  // __CUDACC__

// ---- host-side launch plumbing ------------------------------------------------------------------
struct DeviceInfo {
  int num_sms;
  int max_smem_optin;
};
const DeviceInfo* device_info();  // cached per device; nullptr if the CUDA runtime fails
// Raises a kernel's dynamic shared-memory limit once per (kernel, device); safe from several host threads.
bool configure_kernel_smem(const void* kernel, int bytes);
// Host-side checks of a decode-style call: a coopt_status, nothing is enqueued.
int check_attention_args(const coopt_cache* c, const void* q, void* out, const int32_t* block_table,
                         int32_t max_blocks_per_seq, const int32_t* context_lens, int32_t batch, int32_t num_q_heads);

}  // namespace coopt
