// The decoder (Eq. 5-7) of the separate pass, forward and backward, on the 5th-generation tensor cores: tcgen05.mma
// with the accumulators in tensor memory.  Included by gs_preprocess.cu after the helpers it uses (decoder_inputs,
// load_features, tanh_fast, the mbarrier helpers of namespace bulk).
//
// One CTA of 128 threads works on tiles of 128 Gaussians: thread t owns row t of every operand and lane t of the
// tensor memory.  Per tile and hidden layer the threads write their rows of the A operand (activations, fp16, a high
// and - with split operands - a low half) into shared memory in the canonical K-major layout without swizzle, one
// thread issues the MMAs against the layer's weights (B operand, staged once per CTA) into a 128 x 16 fp32
// accumulator, commits them to an mbarrier, and every thread reads its accumulator row back with tcgen05.ld for
// the ReLU and the next layer; the 3 x 16 output layer runs in registers.  A thread never needs another thread's
// values: no fragment shuffling at all.  The backward (further down) adds the transposed products and takes the
// weight gradients as products over the tile's rows, accumulated in tensor memory.
//
// Single-GPU code: every CTA works alone (no cluster, no copy or commit addressed to more than one CTA).  Every wait
// on the mbarrier is bounded; a wait that runs out sets *timeout (read by gs_async_status), the CTA stops issuing MMAs, runs its loops to the end without
// waiting, frees its tensor memory and returns.
#pragma once

#include "gs_tcgen05.cuh"

namespace tc {

constexpr int kCols = 32;       // columns of tensor memory per CTA: two accumulators of 16 (the output layer's takes the first again)
constexpr int kCtasPerSm = 8;   // what 63 registers x 128 threads allow; 8 x 32 columns and 8 x 19 KB fit the SM

// The output layer (3 x 16 products per Gaussian) in registers, on the fp32 activations: cheaper than a phase of its
// own (operand rows, barrier, MMA round trip, read-back).  w3f = W3 as floats, [3][16].
__device__ __forceinline__ void output_layer(const float *w3f, const float h[16], float y[3]) {
  y[0] = y[1] = y[2] = 0.f;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const float4 r0 = *reinterpret_cast<const float4 *>(w3f + 4 * q), r1 = *reinterpret_cast<const float4 *>(w3f + 16 + 4 * q),
                 r2 = *reinterpret_cast<const float4 *>(w3f + 32 + 4 * q);
    y[0] = fmaf(h[4 * q], r0.x, fmaf(h[4 * q + 1], r0.y, fmaf(h[4 * q + 2], r0.z, fmaf(h[4 * q + 3], r0.w, y[0]))));
    y[1] = fmaf(h[4 * q], r1.x, fmaf(h[4 * q + 1], r1.y, fmaf(h[4 * q + 2], r1.z, fmaf(h[4 * q + 3], r1.w, y[1]))));
    y[2] = fmaf(h[4 * q], r2.x, fmaf(h[4 * q + 1], r2.y, fmaf(h[4 * q + 2], r2.z, fmaf(h[4 * q + 3], r2.w, y[2]))));
  }
}

struct __align__(128) Smem {
  // A operand, high and low halves: 4 K chunks x 128 rows x 16 B for the first layer; the later layers (2 chunks)
  // write over it - their rows are written after the MMAs that read the previous contents have completed
  unsigned char a1[2][4 * kTile * 16];
  unsigned char w1[4 * 16 * 16];         // W1 [16][32] as B operand: 4 K chunks x 16 rows x 16 B
  unsigned char w2[2 * 16 * 16];         // W2 [16][16]
  float w3f[3 * 16];                     // W3 as floats: the output layer runs in registers
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
  }
  for (int idx = tid; idx < 3 * 16; idx += kTile) S.w3f[idx] = __half2float(a.weights[768 + idx]);
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
  const uint32_t A4 = bulk::smem_addr(S.a1[0]) >> 4, W14 = bulk::smem_addr(S.w1) >> 4, W24 = bulk::smem_addr(S.w2) >> 4;
  constexpr int kParts = kSplit ? 2 : 1;
  constexpr uint32_t kPartStride = 4u * chunk_bytes(kTile);      // the low halves' buffer follows the high halves'
  uint32_t phase = 0;

  // one layer: the operands are in shared memory; issue (one thread), commit, wait (bounded)
  auto run_layer = [&](auto issue) {
    bulk::fence_generic_writes();     // the rows just written with ordinary stores, for the tensor core's reads
    fence_before_sync();
    __syncthreads();
    if (tid == 0 && !*reinterpret_cast<volatile uint32_t *>(&S.failed)) {
      fence_after_sync();
      issue();
      commit(bar);
    }
    if (!*reinterpret_cast<volatile uint32_t *>(&S.failed)) {
      if (!wait_phase(bar, phase & 1u)) {
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
      const int64_t nx = i + (int64_t)gridDim.x * kTile;     // this thread's row of the CTA's next tile
      if (nx < a.n) {
        prefetch_l2(a.dirs + 3 * nx); prefetch_l2(a.base_color + 3 * nx);
        prefetch_l2(reinterpret_cast<const uint4 *>(a.features) + nx);
      }
    }
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
    run_layer([&] { rows_times<kParts, 2, 16, kPartStride>(tmem + 0u, A4, W14, idesc(128, 16)); });
    float h[16];
    load16(my_lane + 0u, h);
#pragma unroll
    for (int k = 0; k < 16; ++k) h[k] = fmaxf(h[k], 0.f);
#pragma unroll
    for (int c = 0; c < 2; ++c) store_chunk<kSplit>(S.a1[0], S.a1[1], (uint32_t)c * chunk_bytes(kTile) + (uint32_t)tid * 16u, h + 8 * c);
    run_layer([&] { rows_times<kParts, 1, 16, kPartStride>(tmem + 16u, A4, W24, idesc(128, 16)); });
    load16(my_lane + 16u, h);
#pragma unroll
    for (int k = 0; k < 16; ++k) h[k] = fmaxf(h[k], 0.f);
    float y[3];
    output_layer(S.w3f, h, y);
    if (in)
      store3(a.color, i, color_act_z(a.act, base[0] + 0.5f + tanh_fast(y[0])), color_act_z(a.act, base[1] + 0.5f + tanh_fast(y[1])),
             color_act_z(a.act, base[2] + 0.5f + tanh_fast(y[2])));
  }
  fence_before_sync();
  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)kCols) : "memory");
}

// ---- backward ----------------------------------------------------------------------------------------------------
// Per tile of 128 Gaussians, thread t = row t throughout:
//   P1-P2  the forward again (activations are recomputed, not stored): X -> h1 -> h2, every layer's operand rows
//          staying in shared memory because the weight gradients need them; the output layer y = W3 h2 in registers;
//   gy = dL/dy through the activation and the tanh; delta2 = (gy W3) relu'(h2) in registers (3 x 16 products);
//   P4     delta1_pre = delta2 W2 (B operand: W2 transposed); delta1 = delta1_pre relu'(h1);
//   P5     gx = delta1 W1 (B operand: W1 transposed, N = 32), and in the same batch the three weight gradients as
//          products over the tile's 128 Gaussians (K = 128, eight K steps): dW1^T = X^T delta1, dW2^T = h1^T delta2,
//          dW3^T = h2^T gy.  Their operands are the SAME buffers read MN-major (the row index is K).  The buffers
//          X, h1, h2 (high and low halves each) lie behind one another and so do delta2, delta1, gy: ONE product
//          [X | h1 | h2]^T [delta2 | delta1 | gy] with M = 128 and N = 80 per K step holds the three gradients as
//          blocks (the other blocks are computed and ignored) - a tcgen05.mma costs about the same whatever its N,
//          so eight of these replace forty-eight small ones.  High- and low-half rows and columns are added when the
//          CTA writes its partial.  The accumulator stays in tensor memory across all tiles of the CTA.
//   then   dL/df and dL/dd from gx in registers, as in the warp-level kernel.
// Columns of tensor memory: the chain's accumulators share columns 0..31 (each is read back before the next product
// that writes there is issued: F1 = layer 1 and output layer, F2 = layer 2, E = delta1_pre, GX over both), the weight
// gradients' 128 x 80 block follows.
constexpr int kColsBwd = 128;
constexpr uint32_t kF1 = 0, kF2 = 16, kE = 16, kGX = 0, kDW = 32;
constexpr int kCtasPerSmBwd = 4;   // 57 KB of shared memory, 127 registers and 128 columns each: four fit an SM exactly

struct __align__(128) SmemBwd {
  unsigned char x[2][4 * kTile * 16];    // layer-1 inputs, high then low halves: 8 chunks of 2048 B in a row
  unsigned char h1[2][2 * kTile * 16];   // relu(h1): chunks hi0 hi1 lo0 lo1
  unsigned char h2[2][2 * kTile * 16];
  unsigned char d2[2][2 * kTile * 16];   // delta2
  unsigned char d1[2][2 * kTile * 16];   // delta1
  unsigned char gy[2][1 * kTile * 16];   // dL/dy, 3 of 8 columns used
  unsigned char w1[4 * 16 * 16], w2[2 * 16 * 16];   // B operands of the forward's two hidden layers
  unsigned char w2t[2 * 16 * 16];        // B[n = i][k = j] = W2[j][i]
  unsigned char w1t[2 * 32 * 16];        // B[n = k][kk = i] = W1[i][k], N = 32
  float w3f[3 * 16];                     // W3 as floats for the 3 x 16 products in registers
  unsigned long long bar;
  uint32_t tmem_base;
  uint32_t failed;
};

template <bool kSplit>
__global__ void __launch_bounds__(kTile) k_appearance_bwd_tc(AppearanceArgs a) {
  extern __shared__ __align__(128) unsigned char tc_smem[];
  SmemBwd &S = *reinterpret_cast<SmemBwd *>(tc_smem);
  const int tid = threadIdx.x, warp = tid >> 5;
  for (int idx = tid; idx < 16 * 32; idx += kTile) {
    const int i = idx >> 5, k = idx & 31;
    const __half w = a.weights[idx];
    *reinterpret_cast<__half *>(S.w1 + elem_offset(16, i, k)) = w;
    *reinterpret_cast<__half *>(S.w1t + elem_offset(32, k, i)) = w;
  }
  for (int idx = tid; idx < 16 * 16; idx += kTile) {
    const int j = idx >> 4, i = idx & 15;
    const __half w = a.weights[512 + idx];
    *reinterpret_cast<__half *>(S.w2 + elem_offset(16, j, i)) = w;
    *reinterpret_cast<__half *>(S.w2t + elem_offset(16, i, j)) = w;
  }
  for (int idx = tid; idx < 3 * 16; idx += kTile) S.w3f[idx] = __half2float(a.weights[768 + idx]);
  // the low-half buffers are read as rows of the M = 64 operands even when nothing is written there: start them at zero
  for (int idx = tid; idx < (int)(offsetof(SmemBwd, w1) / 16); idx += kTile) reinterpret_cast<uint4 *>(tc_smem)[idx] = make_uint4(0u, 0u, 0u, 0u);
  const uint32_t bar = bulk::smem_addr(&S.bar);
  if (tid == 0) {
    bulk::barrier_init(bar);
    bulk::fence_barrier_init();
    S.failed = 0u;
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(bulk::smem_addr(&S.tmem_base)), "r"((uint32_t)kColsBwd) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  bulk::fence_generic_writes();
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t *>(&S.tmem_base);
  const uint32_t my_lane = tmem + ((uint32_t)(warp * 32) << 16);
  // address fields (address >> 4) of the operand buffers
  const uint32_t X4 = bulk::smem_addr(S.x[0]) >> 4, H14 = bulk::smem_addr(S.h1[0]) >> 4, H24 = bulk::smem_addr(S.h2[0]) >> 4;
  const uint32_t D24 = bulk::smem_addr(S.d2[0]) >> 4, D14 = bulk::smem_addr(S.d1[0]) >> 4;
  const uint32_t W14 = bulk::smem_addr(S.w1) >> 4, W24 = bulk::smem_addr(S.w2) >> 4;
  const uint32_t W2T4 = bulk::smem_addr(S.w2t) >> 4, W1T4 = bulk::smem_addr(S.w1t) >> 4;
  constexpr int kParts = kSplit ? 2 : 1;
  constexpr uint32_t kChunk = chunk_bytes(kTile);          // 2048
  uint32_t phase = 0;
  bool first_tile = true;

  // One batch of MMAs: `issue` runs in thread 0 only, between the CTA barrier and the commit.
  auto run_phase = [&](auto issue) {
    bulk::fence_generic_writes();
    fence_before_sync();
    __syncthreads();
    if (tid == 0 && !*reinterpret_cast<volatile uint32_t *>(&S.failed)) {
      fence_after_sync();
      issue();
      commit(bar);
    }
    if (!*reinterpret_cast<volatile uint32_t *>(&S.failed)) {
      if (!wait_phase(bar, phase & 1u)) {
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
    const bool exists = i < a.n;
    const bool in = exists && (!a.mask || __ldg(a.mask + i) != 0u);
    float d[3] = {0.f, 0.f, 1.f}, base[3] = {0.f, 0.f, 0.f}, gcol[3] = {0.f, 0.f, 0.f};
    float sc[16];                        // (sin f_j, cos f_j): inputs 16..31, needed again for dL/df
    {
      const int64_t nx = i + (int64_t)gridDim.x * kTile;     // this thread's row of the CTA's next tile
      if (nx < a.n) {
        prefetch_l2(a.dirs + 3 * nx); prefetch_l2(a.base_color + 3 * nx); prefetch_l2(a.g_color + 3 * nx);
        prefetch_l2(reinterpret_cast<const uint4 *>(a.features) + nx);
      }
    }
    {
      float x[32];
      if (in) {
        float f[8];
        load3(a.dirs, i, d);
        load3(a.base_color, i, base);
        load3(a.g_color, i, gcol);
        load_features(a.features, i, f);
        decoder_inputs(d[0], d[1], d[2], f, a.deg, x);
      } else {
#pragma unroll
        for (int k = 0; k < 32; ++k) x[k] = 0.f;
      }
#pragma unroll
      for (int k = 0; k < 16; ++k) sc[k] = x[16 + k];
#pragma unroll
      for (int c = 0; c < 4; ++c) store_chunk<kSplit>(S.x[0], S.x[1], (uint32_t)c * kChunk + (uint32_t)tid * 16u, x + 8 * c);
    }
    run_phase([&] { rows_times<kParts, 2, 16, 4u * kChunk>(tmem + kF1, X4, W14, idesc(128, 16)); });
    float h[16];
    uint32_t m1 = 0u, m2 = 0u;           // relu'(h1), relu'(h2) as bit masks
    load16(my_lane + kF1, h);
#pragma unroll
    for (int k = 0; k < 16; ++k) { m1 |= (h[k] > 0.f ? 1u : 0u) << k; h[k] = fmaxf(h[k], 0.f); }
#pragma unroll
    for (int c = 0; c < 2; ++c) store_chunk<kSplit>(S.h1[0], S.h1[1], (uint32_t)c * kChunk + (uint32_t)tid * 16u, h + 8 * c);
    run_phase([&] { rows_times<kParts, 1, 16, 2u * kChunk>(tmem + kF2, H14, W24, idesc(128, 16)); });
    load16(my_lane + kF2, h);
#pragma unroll
    for (int k = 0; k < 16; ++k) { m2 |= (h[k] > 0.f ? 1u : 0u) << k; h[k] = fmaxf(h[k], 0.f); }
#pragma unroll
    for (int c = 0; c < 2; ++c) store_chunk<kSplit>(S.h2[0], S.h2[1], (uint32_t)c * kChunk + (uint32_t)tid * 16u, h + 8 * c);
    float gp[3], gy[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    {
      float y[3];
      output_layer(S.w3f, h, y);
#pragma unroll
      for (int c = 0; c < 3; ++c) {
        const float A = tanh_fast(y[c]);
        gp[c] = in ? color_act_grad_z(a.act, base[c] + 0.5f + A) * gcol[c] : 0.f;
        gy[c] = gp[c] * (1.f - A * A);
      }
    }
    store_chunk<kSplit>(S.gy[0], S.gy[1], (uint32_t)tid * 16u, gy);
    // delta2 = (gy W3) relu'(h2)
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const float4 r0 = *reinterpret_cast<const float4 *>(S.w3f + 4 * q), r1 = *reinterpret_cast<const float4 *>(S.w3f + 16 + 4 * q),
                   r2 = *reinterpret_cast<const float4 *>(S.w3f + 32 + 4 * q);
      h[4 * q] = fmaf(gy[0], r0.x, fmaf(gy[1], r1.x, gy[2] * r2.x));
      h[4 * q + 1] = fmaf(gy[0], r0.y, fmaf(gy[1], r1.y, gy[2] * r2.y));
      h[4 * q + 2] = fmaf(gy[0], r0.z, fmaf(gy[1], r1.z, gy[2] * r2.z));
      h[4 * q + 3] = fmaf(gy[0], r0.w, fmaf(gy[1], r1.w, gy[2] * r2.w));
    }
#pragma unroll
    for (int k = 0; k < 16; ++k) h[k] = (m2 >> k) & 1u ? h[k] : 0.f;
#pragma unroll
    for (int c = 0; c < 2; ++c) store_chunk<kSplit>(S.d2[0], S.d2[1], (uint32_t)c * kChunk + (uint32_t)tid * 16u, h + 8 * c);
    run_phase([&] { rows_times<kParts, 1, 16, 2u * kChunk>(tmem + kE, D24, W2T4, idesc(128, 16)); });
    load16(my_lane + kE, h);
#pragma unroll
    for (int k = 0; k < 16; ++k) h[k] = (m1 >> k) & 1u ? h[k] : 0.f;
#pragma unroll
    for (int c = 0; c < 2; ++c) store_chunk<kSplit>(S.d1[0], S.d1[1], (uint32_t)c * kChunk + (uint32_t)tid * 16u, h + 8 * c);
    const bool fresh = first_tile;
    run_phase([&] {
      rows_times<kParts, 1, 32, 2u * kChunk>(tmem + kGX, D14, W1T4, idesc(128, 32));
      // weight gradients: K runs over the tile's rows, 16 per MMA; A = [X | h1 | h2] (16 chunks), B = [delta2 | delta1 | gy] (10)
#pragma unroll
      for (int ks = 0; ks < kTile / 16; ++ks)
        mma(tmem + kDW, desc_at<128u, kChunk>(X4, (uint32_t)ks * 256u), desc_at<128u, kChunk>(D24, (uint32_t)ks * 256u),
            (fresh && ks == 0) ? 0u : 1u, idesc(128, 80, true, true));
    });
    first_tile = false;
    float gx[32];
    load16(my_lane + kGX, gx);
    load16(my_lane + kGX + 16u, gx + 16);
    if (exists) {
      float gf[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) gf[j] = gx[16 + 2 * j] * sc[2 * j + 1] - gx[17 + 2 * j] * sc[2 * j];
      const int na = (a.deg + 1) * (a.deg + 1);
      float ax = 0.f, ay = 0.f, az = 0.f;
#pragma unroll
      for (int k = 1; k < 16; ++k)
        if (k < na) sh_grad_acc(k, d[0], d[1], d[2], gx[k], ax, ay, az);
      float4 *gfp = reinterpret_cast<float4 *>(a.g_features) + 2 * i;
      gfp[0] = make_float4(gf[0], gf[1], gf[2], gf[3]);
      gfp[1] = make_float4(gf[4], gf[5], gf[6], gf[7]);
      store3(a.g_base, i, gp[0], gp[1], gp[2]);
      store3(a.g_dirs, i, ax, ay, az);
    }
  }
  // ---- this CTA's partial of the weight gradient.  Thread t holds row t of the 128 x 80 block: rows 0..63 = X (high,
  // low), 64..95 = h1, 96..127 = h2; columns 0..31 = delta2 (high, low), 32..63 = delta1, 64..79 = gy (8 + 8).
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  float *tmp = reinterpret_cast<float *>(S.x[0]);         // [128][16]: each row's own block, high + low columns added
  {
    float lo[16], hi[16];
    const uint32_t c0 = tid < 64 ? 32u : tid < 96 ? 0u : 64u;     // first column of this row's block
    load16(my_lane + kDW + c0, lo);
    if (tid < 96) {
      load16(my_lane + kDW + c0 + 16u, hi);
#pragma unroll
      for (int k = 0; k < 16; ++k) lo[k] += hi[k];
    } else {
#pragma unroll
      for (int k = 0; k < 8; ++k) lo[k] += lo[8 + k];
    }
#pragma unroll
    for (int k = 0; k < 16; ++k) tmp[tid * 16 + k] = first_tile ? 0.f : lo[k];
  }
  __syncthreads();
  float *out = a.w_partials + (size_t)blockIdx.x * GS_MLP_WEIGHTS;
  for (int idx = tid; idx < 16 * 32; idx += kTile) {      // dW1[i][k] = rows k (high) and 32 + k (low), column i
    const int i = idx >> 5, k = idx & 31;
    out[idx] = tmp[k * 16 + i] + tmp[(32 + k) * 16 + i];
  }
  for (int idx = tid; idx < 16 * 16; idx += kTile) {      // dW2[j][i] = rows i (high) and 16 + i (low), column j
    const int j = idx >> 4, i = idx & 15;
    out[512 + idx] = tmp[(64 + i) * 16 + j] + tmp[(80 + i) * 16 + j];
  }
  for (int idx = tid; idx < 3 * 16; idx += kTile) {       // dW3[c][j] = rows j (high) and 16 + j (low), column c
    const int c = idx >> 4, j = idx & 15;
    out[768 + idx] = tmp[(96 + j) * 16 + c] + tmp[(112 + j) * 16 + c];
  }
  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)kColsBwd) : "memory");
}

}  // namespace tc
