// tcgen05 building blocks shared by the decoder kernels on the 5th-generation tensor cores: instruction and
// shared-memory descriptors for operands in the canonical layouts without swizzle, the MMA / commit / tensor-memory
// load wrappers, the bounded mbarrier wait and the operand-row writer with high / low fp16 halves.  Included inside
// namespace gs's unnamed namespace by the translation units that hold such kernels.  Single-GPU code: every CTA
// works alone (no cluster, no copy or commit addressed to more than one CTA).
#pragma once
#include <cuda_fp16.h>
#include <stdint.h>

namespace tc {

constexpr int kTile = 128;      // Gaussians per tile = rows of an MMA = lanes of tensor memory
// Instruction descriptor of kind::f16: D fp32 (bits 4-5 = 1), A and B fp16 (0), A / B MN-major (bits 15 / 16; 0 =
// K-major), N (bits 17-22 = N >> 3), M (bits 24-28 = M >> 4), dense, no negation.
__host__ __device__ constexpr uint32_t idesc(int m, int n, bool a_mn = false, bool b_mn = false) {
  return (1u << 4) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// Canonical K-major operand without swizzle: core matrices of 8 rows x 16 bytes (8 halves), stored as 128
// contiguous bytes; the core matrices of consecutive 8-row groups lie 128 B apart (stride byte offset), those of
// consecutive 8-element K chunks rows / 8 * 128 B apart (leading byte offset).  Element (row r, column k).
__device__ __forceinline__ constexpr uint32_t chunk_bytes(int rows) { return (uint32_t)rows * 16u; }
__device__ __forceinline__ constexpr uint32_t elem_offset(int rows, int r, int k) {
  return (uint32_t)(k >> 3) * chunk_bytes(rows) + (uint32_t)r * 16u + (uint32_t)(k & 7) * 2u;
}
// Shared-memory matrix descriptor (64 bits): start address (bits 0-13), leading byte offset (16-29) and stride byte
// offset (32-45), all in units of 16 B; descriptor version 1 (bits 46-47); base offset 0; no swizzle (bits 61-63 = 0).
// K-major operand of R rows: leading byte offset = R * 16 (next 8-element K chunk), stride byte offset = 128 (next
// group of 8 rows).  The same buffer read MN-major (the rows are the K dimension, the 16-byte chunks of a row are 8
// consecutive elements of M or N): leading byte offset = 128 (next group of 8 rows of K), stride byte offset = the
// distance of the chunks (next 8 elements of M or N).
// Bounded wait for a phase of the MMAs' mbarrier: the MMAs of a phase complete within a microsecond, so the threads
// poll, with a short pause between polls that leaves the issue slots to the CTAs that have work; 2^22 polls (about a
// second) is the bound after which the caller gives up and reports.
__device__ __forceinline__ bool wait_phase(uint32_t bar, uint32_t parity) {
  for (int it = 0; it < (1 << 22); ++it) {
    uint32_t done;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    if (done) return true;
    __nanosleep(20);
  }
  return false;
}

// The inputs of this thread's row in the tile after the next barrier-bound stretch: asked into L2 ahead of time.
__device__ __forceinline__ void prefetch_l2(const void *p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

__device__ __forceinline__ void mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t accumulate, uint32_t desc);

// The issuing thread's fast path: with the buffer's address field (address >> 4) computed once, a descriptor `off`
// bytes into the buffer is one add (the low word) and an immediate (the high word).  Shared-memory addresses stay
// below 2^18, so the address field never carries into the offset fields.
template <uint32_t kLboBytes, uint32_t kSboBytes>
__device__ __forceinline__ uint64_t desc_at(uint32_t base4, uint32_t off_bytes) {
  const uint32_t lo = base4 + ((off_bytes >> 4) | ((kLboBytes >> 4) << 16));
  constexpr uint32_t hi = (kSboBytes >> 4) | (1u << 14);
  return ((uint64_t)hi << 32) | lo;
}
// D (128 x n) = or += A * B^T for a K-major A of the tile's rows (kSteps x 16 columns per part, kParts parts
// kPartStride bytes apart) and a K-major B of kBRows rows; a4 / b4 are the buffers' address fields.
template <int kParts, int kSteps, int kBRows, uint32_t kPartStride>
__device__ __forceinline__ void rows_times(uint32_t d_tmem, uint32_t a4, uint32_t b4, uint32_t desc) {
#pragma unroll
  for (int p = 0; p < kParts; ++p)
#pragma unroll
    for (int ks = 0; ks < kSteps; ++ks)
      mma(d_tmem, desc_at<chunk_bytes(kTile), 128u>(a4, (uint32_t)p * kPartStride + (uint32_t)ks * 2u * chunk_bytes(kTile)),
          desc_at<chunk_bytes(kBRows), 128u>(b4, (uint32_t)ks * 2u * chunk_bytes(kBRows)), (p | ks) ? 1u : 0u, desc);
}

__device__ __forceinline__ void fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D (tensor memory, 128 lanes x 16 columns) = or += A (128 x 16, shared) * B^T (16 x 16, shared); one thread issues.
__device__ __forceinline__ void mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t accumulate, uint32_t desc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(desc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u)
      : "memory");
}
// The mbarrier gets one arrival when every MMA issued so far by this thread has completed.
__device__ __forceinline__ void commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// This thread's lane of the accumulator: 16 consecutive fp32 columns, complete when the call returns.
__device__ __forceinline__ void load16(uint32_t taddr, float v[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
#pragma unroll
  for (int k = 0; k < 16; ++k) v[k] = __uint_as_float(r[k]);
}
// Eight consecutive values of this thread's operand row as one 16-byte chunk of halves: the high halves, and the
// halves of what the rounding left (the products then carry about 22 bits).
template <bool kSplit>
__device__ __forceinline__ void store_chunk(unsigned char *hi, unsigned char *lo, uint32_t offset, const float *v) {
  uint4 h, l;
  uint32_t *hw = reinterpret_cast<uint32_t *>(&h), *lw = reinterpret_cast<uint32_t *>(&l);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const __half2 a = __floats2half2_rn(v[2 * j], v[2 * j + 1]);
    hw[j] = *reinterpret_cast<const uint32_t *>(&a);
    if (kSplit) {
      const float2 f = __half22float2(a);
      const __half2 b = __floats2half2_rn(v[2 * j] - f.x, v[2 * j + 1] - f.y);
      lw[j] = *reinterpret_cast<const uint32_t *>(&b);
    }
  }
  *reinterpret_cast<uint4 *>(hi + offset) = h;
  if (kSplit) *reinterpret_cast<uint4 *>(lo + offset) = l;
}

// Shared-memory address, mbarrier set-up (one arrival) and the fence that makes ordinary shared-memory stores visible
// to the tensor core's reads.
__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void barrier_init(uint32_t bar) { asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar) : "memory"); }
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_generic_writes() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// Tensor-memory columns of the CTA (a power of two >= 32): one warp allocates, the address lands in shared memory;
// the permit is given back at once so that other CTAs of the SM can allocate.  The same warp frees them.
__device__ __forceinline__ void tmem_alloc(uint32_t *slot, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(slot)), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_free(uint32_t tmem, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(cols) : "memory");
}

}  // namespace tc
