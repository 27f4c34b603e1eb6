// The decoder (Eq. 5-7) of the separate-pass forward on the 5th-generation tensor cores: tcgen05.mma with the
// accumulators in tensor memory.  Included by gs_preprocess.cu after the helpers it uses (decoder_inputs,
// load_features, tanh_fast, the bounded mbarrier wait of namespace bulk).
//
// One CTA of 128 threads works on tiles of 128 Gaussians: thread t owns row t of every operand and lane t of the
// tensor memory.  Per tile and layer the threads write their rows of the A operand (activations, fp16, a high and
// - with split operands - a low half) into shared memory in the canonical K-major layout without swizzle, one
// thread issues the MMAs against the layer's weights (B operand, staged once per CTA) into a 128 x 16 fp32
// accumulator, commits them to an mbarrier, and every thread reads its accumulator row back with tcgen05.ld for
// the ReLU and the next layer.  A thread never needs another thread's values: no fragment shuffling at all.
//
// Single-GPU code: no cluster, no multicast of any kind.  Every wait on the mbarrier is bounded; a wait that runs
// out sets *timeout (read by gs_async_status), the CTA stops issuing MMAs, runs its loops to the end without
// waiting, frees its tensor memory and returns.
#pragma once

namespace tc {

constexpr int kTile = 128;      // Gaussians per tile = rows of an MMA = lanes of tensor memory
constexpr int kCols = 32;       // columns of tensor memory per CTA: two accumulators of 16 (the output layer's takes the first again)
constexpr int kCtasPerSm = 8;   // what 63 registers x 128 threads allow; 8 x 32 columns and 8 x 19 KB fit the SM
// Instruction descriptor of kind::f16: D fp32 (bits 4-5 = 1), A and B fp16 (0), both K-major (bits 15, 16 = 0),
// N = 16 (bits 17-22 = N >> 3), M = 128 (bits 24-28 = M >> 4), dense, no negation.
constexpr uint32_t kIdesc = (1u << 4) | ((16u >> 3) << 17) | ((128u >> 4) << 24);

// Canonical K-major operand without swizzle: core matrices of 8 rows x 16 bytes (8 halves), stored as 128
// contiguous bytes; the core matrices of consecutive 8-row groups lie 128 B apart (stride byte offset), those of
// consecutive 8-element K chunks rows / 8 * 128 B apart (leading byte offset).  Element (row r, column k).
__device__ __forceinline__ constexpr uint32_t chunk_bytes(int rows) { return (uint32_t)rows * 16u; }
__device__ __forceinline__ constexpr uint32_t elem_offset(int rows, int r, int k) {
  return (uint32_t)(k >> 3) * chunk_bytes(rows) + (uint32_t)r * 16u + (uint32_t)(k & 7) * 2u;
}
// Shared-memory matrix descriptor: start address, leading and stride byte offsets in units of 16 B, descriptor
// version 1 (bits 46-47), base offset 0, no swizzle (bits 61-63 = 0).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, int rows) {
  return (uint64_t)((addr >> 4) & 0x3fffu) | ((uint64_t)((chunk_bytes(rows) >> 4) & 0x3fffu) << 16) |
         ((uint64_t)(128u >> 4) << 32) | (1ull << 46);
}

__device__ __forceinline__ void fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D (tensor memory, 128 lanes x 16 columns) = or += A (128 x 16, shared) * B^T (16 x 16, shared); one thread issues.
__device__ __forceinline__ void mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(kIdesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u)
      : "memory");
}
// The mbarrier gets one arrival when every MMA issued so far by this thread has completed.
__device__ __forceinline__ void commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// This thread's lane of the accumulator: 16 (or 4) consecutive fp32 columns, complete when the call returns.
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
__device__ __forceinline__ void load4(uint32_t taddr, float v[4]) {
  uint32_t r[4];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
      : "r"(taddr)
      : "memory");
#pragma unroll
  for (int k = 0; k < 4; ++k) v[k] = __uint_as_float(r[k]);
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

struct __align__(128) Smem {
  // A operand, high and low halves: 4 K chunks x 128 rows x 16 B for the first layer; the later layers (2 chunks)
  // write over it - their rows are written after the MMAs that read the previous contents have completed
  unsigned char a1[2][4 * kTile * 16];
  unsigned char w1[4 * 16 * 16];         // W1 [16][32] as B operand: 4 K chunks x 16 rows x 16 B
  unsigned char w2[2 * 16 * 16];         // W2 [16][16]
  unsigned char w3[2 * 16 * 16];         // W3 [3][16], rows 3..15 zero
  unsigned long long bar;
  uint32_t tmem_base;
  uint32_t failed;
};

template <bool kSplit>
__global__ void __launch_bounds__(kTile) k_appearance_fwd_tc(AppearanceArgs a) {
  extern __shared__ __align__(128) unsigned char tc_smem[];
  Smem &S = *reinterpret_cast<Smem *>(tc_smem);
  const int tid = threadIdx.x, warp = tid >> 5;
  // weights into the B-operand layout (row = output neuron, K = input), once per CTA
  for (int idx = tid; idx < 16 * 32; idx += kTile) {
    const int n = idx >> 5, k = idx & 31;
    *reinterpret_cast<__half *>(S.w1 + elem_offset(16, n, k)) = a.weights[idx];
  }
  for (int idx = tid; idx < 16 * 16; idx += kTile) {
    const int n = idx >> 4, k = idx & 15;
    *reinterpret_cast<__half *>(S.w2 + elem_offset(16, n, k)) = a.weights[512 + idx];
    *reinterpret_cast<__half *>(S.w3 + elem_offset(16, n, k)) = n < 3 ? a.weights[768 + idx] : __float2half(0.f);
  }
  const uint32_t bar = bulk::smem_addr(&S.bar);
  if (tid == 0) {
    bulk::barrier_init(bar);
    bulk::fence_barrier_init();
    S.failed = 0u;
  }
  if (warp == 0) {   // one warp allocates the CTA's columns of tensor memory and gives the permit back at once
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(bulk::smem_addr(&S.tmem_base)), "r"((uint32_t)kCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  bulk::fence_generic_writes();
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t *>(&S.tmem_base);
  const uint32_t my_lane = tmem + ((uint32_t)(warp * 32) << 16);   // this warp's 32 lanes (bits 16..31 of the address)
  const uint32_t A1[2] = {bulk::smem_addr(S.a1[0]), bulk::smem_addr(S.a1[1])};
  const uint32_t W1 = bulk::smem_addr(S.w1), W2 = bulk::smem_addr(S.w2), W3 = bulk::smem_addr(S.w3);
  constexpr int kParts = kSplit ? 2 : 1;
  uint32_t phase = 0;

  // one layer: the operands are in shared memory; issue, commit, wait (bounded)
  auto run_layer = [&](const uint32_t A[2], uint32_t W, int ksteps, uint32_t d_cols) {
    bulk::fence_generic_writes();     // the rows just written with ordinary stores, for the tensor core's reads
    fence_before_sync();
    __syncthreads();
    if (tid == 0 && !*reinterpret_cast<volatile uint32_t *>(&S.failed)) {
      fence_after_sync();
      uint32_t acc = 0u;
      for (int p = 0; p < kParts; ++p)
        for (int ks = 0; ks < ksteps; ++ks) {   // 16 columns of K per MMA = two chunks
          mma(tmem + d_cols, smem_desc(A[p] + (uint32_t)ks * 2u * chunk_bytes(kTile), kTile),
              smem_desc(W + (uint32_t)ks * 2u * chunk_bytes(16), 16), acc);
          acc = 1u;
        }
      commit(bar);
    }
    if (!*reinterpret_cast<volatile uint32_t *>(&S.failed)) {
      if (!bulk::wait(bar, phase & 1u)) {
        S.failed = 1u;
        if (a.timeout) atomicExch(a.timeout, 1ull);
      }
    }
    ++phase;
    fence_after_sync();
  };

  const int64_t ntiles = (a.n + kTile - 1) / kTile;
  for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
    const int64_t i = tile * kTile + tid;
    const bool in = i < a.n && (!a.mask || __ldg(a.mask + i) != 0u);
    float base[3] = {0.f, 0.f, 0.f};
    {
      float x[32];
      if (in) {
        float d[3], f[8];
        load3(a.dirs, i, d);
        load3(a.base_color, i, base);
        load_features(a.features, i, f);
        decoder_inputs(d[0], d[1], d[2], f, a.deg, x);
      } else {
#pragma unroll
        for (int k = 0; k < 32; ++k) x[k] = 0.f;
      }
#pragma unroll
      for (int c = 0; c < 4; ++c) store_chunk<kSplit>(S.a1[0], S.a1[1], (uint32_t)c * chunk_bytes(kTile) + (uint32_t)tid * 16u, x + 8 * c);
    }
    run_layer(A1, W1, 2, 0u);
    float h[16];
    load16(my_lane + 0u, h);
#pragma unroll
    for (int k = 0; k < 16; ++k) h[k] = fmaxf(h[k], 0.f);
#pragma unroll
    for (int c = 0; c < 2; ++c) store_chunk<kSplit>(S.a1[0], S.a1[1], (uint32_t)c * chunk_bytes(kTile) + (uint32_t)tid * 16u, h + 8 * c);
    run_layer(A1, W2, 1, 16u);
    load16(my_lane + 16u, h);
#pragma unroll
    for (int k = 0; k < 16; ++k) h[k] = fmaxf(h[k], 0.f);
#pragma unroll
    for (int c = 0; c < 2; ++c) store_chunk<kSplit>(S.a1[0], S.a1[1], (uint32_t)c * chunk_bytes(kTile) + (uint32_t)tid * 16u, h + 8 * c);
    run_layer(A1, W3, 1, 0u);
    float y[4];
    load4(my_lane + 0u, y);
    if (in)
      store3(a.color, i, color_act_z(a.act, base[0] + 0.5f + tanh_fast(y[0])), color_act_z(a.act, base[1] + 0.5f + tanh_fast(y[1])),
             color_act_z(a.act, base[2] + 0.5f + tanh_fast(y[2])));
  }
  fence_before_sync();
  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)kCols) : "memory");
}

}  // namespace tc
