// The decoder variants of the architecture table (App. D: 1 to 3 hidden layers of 16 or 32 neurons, 8 frequency-
// encoded or 16 raw features) on the 5th-generation tensor cores.  Included by gs_decoder_variants.cu after VarDims
// and variant_inputs.  Same scheme as the default decoder's tcgen05 kernels, generalised over the layer shapes:
//
// One CTA of 128 threads works on tiles of 128 Gaussians; thread t owns row t of every operand and lane t of tensor
// memory.  Per tile and hidden layer the threads write their rows of the A operand (fp16, a high and a low half, so
// that the products carry about 22 bits) in the canonical K-major layout, one thread issues the MMAs against the
// layer's weights (B operand, staged once per CTA) into a 128 x H fp32 accumulator, commits them to an mbarrier, and
// every thread reads its accumulator row back for the ReLU; the 3 x H output layer runs in registers.
//
// The backward runs the forward again, keeps every layer's operand rows in shared memory, takes the transposed
// products layer by layer, and forms all weight gradients as products over the tile's rows: the operand buffers
// [X | h_1 | ... | h_L] lie behind one another and so do [delta_1 | ... | delta_L | gy], and each block of 128
// columns of the first, read MN-major, is multiplied with the range of the second that holds its partners (W_1
// pairs X with delta_1, W_(l+1) pairs h_l with delta_(l+1), W_out pairs h_L with gy).  A tcgen05.mma costs about the
// same whatever its N, so one or two wide products per 16 Gaussians replace a dozen small ones; the blocks that pair
// non-partners are computed and ignored.  The accumulators stay in tensor memory across all tiles of the CTA.
//
// Single-GPU code: every CTA works alone (no cluster).  Every wait is bounded; one that runs out sets *timeout (read by
// gs_async_status), the CTA stops issuing MMAs, runs its loops to the end without waiting, frees its tensor memory
// and returns.
#pragma once

#include "gs_tcgen05.cuh"

namespace vtc {

constexpr uint32_t kChunk = tc::chunk_bytes(tc::kTile);   // 2048 B: 128 rows x 8 halves

template <int H, int L>
struct Shape {
  static constexpr int kHC = H / 8;                       // 16-byte chunks of a hidden operand row
  static constexpr int kHS = H / 16;                      // K steps of a product over a hidden layer
  // buffers of the backward, in chunks of 2048 B; every buffer holds its high halves, then its low halves
  static constexpr int kAChunks = 8 + L * 2 * kHC;        // X (4 + 4), h_1 .. h_L
  static constexpr int kBChunks = L * 2 * kHC + 2;        // delta_1 .. delta_L, gy (1 + 1)
  static constexpr int kBlocks = (kAChunks + 15) / 16;    // blocks of 128 columns of [X | h_1 | ...]
  __host__ __device__ static constexpr int a_start(int j) { return j == 0 ? 0 : 8 + (j - 1) * 2 * kHC; }   // j = 0: X, j: h_j
  __host__ __device__ static constexpr int a_len(int j) { return j == 0 ? 8 : 2 * kHC; }
  __host__ __device__ static constexpr int b_start(int j) { return j * 2 * kHC; }                          // partner of a-buffer j
  __host__ __device__ static constexpr int b_len(int j) { return j < L ? 2 * kHC : 2; }
  // the a-buffers that block b holds (no buffer straddles two blocks: 64 and 2 H divide 128)
  __host__ __device__ static constexpr int first_buffer(int b) {
    int j = 0;
    while (a_start(j) + a_len(j) <= 16 * b) ++j;
    return j;
  }
  __host__ __device__ static constexpr int last_buffer(int b) {
    int j = L;
    while (a_start(j) >= 16 * b + 16) --j;
    return j;
  }
  __host__ __device__ static constexpr int n_start(int b) { return b_start(first_buffer(b)); }             // chunks
  __host__ __device__ static constexpr int n_cols(int b) { return 8 * (b_start(last_buffer(b)) + b_len(last_buffer(b)) - n_start(b)); }
  __host__ __device__ static constexpr int dw_col(int b) { return b == 0 ? 0 : dw_col(b - 1) + n_cols(b - 1); }
  // columns of tensor memory: the chain's accumulators share columns 0..31 (each is read back before the next
  // product that writes there is issued), the weight-gradient blocks follow
  // (dL/dx, 32 wide, is then taken in two halves of 16, one phase each: worth it where it halves the allocation)
  static constexpr bool kSplitGx = H == 16 && 32 + dw_col(kBlocks) > 128 && 16 + dw_col(kBlocks) <= 128;
  static constexpr int kChainCols = kSplitGx ? 16 : 32;
  static constexpr int kColsUsed = kChainCols + dw_col(kBlocks);
  static constexpr int kColsAlloc = kColsUsed <= 32 ? 32 : kColsUsed <= 64 ? 64 : kColsUsed <= 128 ? 128 : kColsUsed <= 256 ? 256 : 512;
  static_assert(H == 16 || H == 32, "hidden width");
  static_assert(L >= 1 && L <= 3, "hidden layers");
  static_assert(kColsUsed <= 512, "tensor memory");
};

// Inputs of one Gaussian: the default decoder's (fast sine / cosine inside [-pi, pi]) for 8 encoded features, the SH
// basis followed by the 16 raw features otherwise.
__device__ __forceinline__ void inputs(const AppearanceArgs &a, int64_t i, int nfeat, const float d[3], float x[32]) {
  if (nfeat == 8) {
    float f[8];
    load_features(a.features, i, f);
    decoder_inputs(d[0], d[1], d[2], f, a.deg, x);
  } else {
    variant_inputs(a, i, nfeat, d, x);
  }
}

template <int H>
__device__ __forceinline__ void load_row(uint32_t taddr, float *v) {
#pragma unroll
  for (int q = 0; q < H / 16; ++q) tc::load16(taddr + 16u * q, v + 16 * q);
}
template <int H>
__device__ __forceinline__ void store_row(unsigned char *buf, int tid, const float *v) {   // high halves, then low halves
#pragma unroll
  for (int c = 0; c < H / 8; ++c) tc::store_chunk<true>(buf, buf + (H / 8) * kChunk, (uint32_t)c * kChunk + (uint32_t)tid * 16u, v + 8 * c);
}
// y = W_out h in registers: wf = W_out as floats, [3][H]
template <int H>
__device__ __forceinline__ void output_layer(const float *wf, const float *h, float y[3]) {
  y[0] = y[1] = y[2] = 0.f;
#pragma unroll
  for (int q = 0; q < H / 4; ++q) {
    const float4 r0 = *reinterpret_cast<const float4 *>(wf + 4 * q), r1 = *reinterpret_cast<const float4 *>(wf + H + 4 * q),
                 r2 = *reinterpret_cast<const float4 *>(wf + 2 * H + 4 * q);
    y[0] = fmaf(h[4 * q], r0.x, fmaf(h[4 * q + 1], r0.y, fmaf(h[4 * q + 2], r0.z, fmaf(h[4 * q + 3], r0.w, y[0]))));
    y[1] = fmaf(h[4 * q], r1.x, fmaf(h[4 * q + 1], r1.y, fmaf(h[4 * q + 2], r1.z, fmaf(h[4 * q + 3], r1.w, y[1]))));
    y[2] = fmaf(h[4 * q], r2.x, fmaf(h[4 * q + 1], r2.y, fmaf(h[4 * q + 2], r2.z, fmaf(h[4 * q + 3], r2.w, y[2]))));
  }
}

// Weights into the B-operand layouts (row = output index of the product, K = the index summed over), once per CTA.
// w1: W_1 [H][32]; wl[l]: W_(l+2) [H][H]; the transposed forms for the backward's products.
template <int H, int L>
__device__ __forceinline__ void stage_weights(const __half *w, unsigned char *w1, unsigned char *wl, float *woutf, unsigned char *w1t,
                                              unsigned char *wlt, int tid) {
  for (int idx = tid; idx < H * 32; idx += tc::kTile) {
    const int i = idx >> 5, k = idx & 31;
    const __half v = w[idx];
    *reinterpret_cast<__half *>(w1 + tc::elem_offset(H, i, k)) = v;
    if (w1t) *reinterpret_cast<__half *>(w1t + tc::elem_offset(32, k, i)) = v;
  }
  for (int l = 1; l < L; ++l)
    for (int idx = tid; idx < H * H; idx += tc::kTile) {
      const int j = idx / H, i = idx % H;
      const __half v = w[VarDims<H, L>::off(l) + idx];
      *reinterpret_cast<__half *>(wl + (l - 1) * 2 * H * H + tc::elem_offset(H, j, i)) = v;
      if (wlt) *reinterpret_cast<__half *>(wlt + (l - 1) * 2 * H * H + tc::elem_offset(H, i, j)) = v;
    }
  for (int idx = tid; idx < 3 * H; idx += tc::kTile) woutf[idx] = __half2float(w[VarDims<H, L>::off(L) + idx]);
}

template <int H, int L>
struct __align__(128) SmemFwd {
  unsigned char a[2][4 * tc::kTile * 16];          // A operand, high and low halves: 4 K chunks for the first layer, H / 8 after
  unsigned char w1[4 * H * 16];
  unsigned char wl[(L > 1 ? L - 1 : 1) * 2 * H * H];
  float woutf[3 * H];
  unsigned long long bar;
  uint32_t tmem_base;
  uint32_t failed;
};

template <int H, int L>
__global__ void __launch_bounds__(tc::kTile) k_variant_fwd_tc(AppearanceArgs a, int nfeat) {
  using S_t = SmemFwd<H, L>;
  using Sh = Shape<H, L>;
  extern __shared__ __align__(128) unsigned char vtc_smem[];
  S_t &S = *reinterpret_cast<S_t *>(vtc_smem);
  const int tid = threadIdx.x, warp = tid >> 5;
  stage_weights<H, L>(a.weights, S.w1, S.wl, S.woutf, nullptr, nullptr, tid);
  const uint32_t bar = tc::smem_addr(&S.bar);
  if (tid == 0) {
    tc::barrier_init(bar);
    tc::fence_barrier_init();
    S.failed = 0u;
  }
  if (warp == 0) tc::tmem_alloc(&S.tmem_base, 32u);
  tc::fence_generic_writes();
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t *>(&S.tmem_base);
  const uint32_t my_lane = tmem + ((uint32_t)(warp * 32) << 16);
  const uint32_t A4 = tc::smem_addr(S.a[0]) >> 4, W14 = tc::smem_addr(S.w1) >> 4, WL4 = tc::smem_addr(S.wl) >> 4;
  uint32_t phase = 0;
  auto run_layer = [&](auto issue) {
    tc::fence_generic_writes();
    tc::fence_before_sync();
    __syncthreads();
    if (tid == 0 && !*reinterpret_cast<volatile uint32_t *>(&S.failed)) {
      tc::fence_after_sync();
      issue();
      tc::commit(bar);
    }
    if (!*reinterpret_cast<volatile uint32_t *>(&S.failed)) {
      if (!tc::wait_phase(bar, phase & 1u)) {
        S.failed = 1u;
        if (a.timeout) atomicExch(a.timeout, 1ull);
      }
    }
    ++phase;
    tc::fence_after_sync();
  };
  const int64_t ntiles = (a.n + tc::kTile - 1) / tc::kTile;
  for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
    const int64_t i = tile * tc::kTile + tid;
    const bool in = i < a.n && (!a.mask || __ldg(a.mask + i) != 0u);
    float base[3] = {0.f, 0.f, 0.f};
    {
      float x[32];
      if (in) {
        float d[3];
#pragma unroll
        for (int c = 0; c < 3; ++c) { d[c] = __ldg(a.dirs + 3 * i + c); base[c] = __ldg(a.base_color + 3 * i + c); }
        inputs(a, i, nfeat, d, x);
      } else {
#pragma unroll
        for (int k = 0; k < 32; ++k) x[k] = 0.f;
      }
#pragma unroll
      for (int c = 0; c < 4; ++c) tc::store_chunk<true>(S.a[0], S.a[1], (uint32_t)c * kChunk + (uint32_t)tid * 16u, x + 8 * c);
    }
    run_layer([&] { tc::rows_times<2, 2, H, 4u * kChunk>(tmem, A4, W14, tc::idesc(128, H)); });
    float h[H];
    load_row<H>(my_lane, h);
#pragma unroll
    for (int k = 0; k < H; ++k) h[k] = fmaxf(h[k], 0.f);
#pragma unroll
    for (int l = 1; l < L; ++l) {
#pragma unroll
      for (int c = 0; c < Sh::kHC; ++c) tc::store_chunk<true>(S.a[0], S.a[1], (uint32_t)c * kChunk + (uint32_t)tid * 16u, h + 8 * c);
      run_layer([&] { tc::rows_times<2, Sh::kHS, H, 4u * kChunk>(tmem, A4, WL4 + (uint32_t)((l - 1) * 2 * H * H >> 4), tc::idesc(128, H)); });
      load_row<H>(my_lane, h);
#pragma unroll
      for (int k = 0; k < H; ++k) h[k] = fmaxf(h[k], 0.f);
    }
    float y[3];
    output_layer<H>(S.woutf, h, y);
    if (in) {
#pragma unroll
      for (int c = 0; c < 3; ++c) a.color[3 * i + c] = color_act_z(a.act, base[c] + 0.5f + tanh_fast(y[c]));
    }
  }
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 0) tc::tmem_free(tmem, 32u);
}

template <int H, int L>
struct __align__(128) SmemBwd {
  unsigned char a[Shape<H, L>::kAChunks * kChunk];   // [X | h_1 | ... | h_L], each high halves then low halves
  unsigned char b[Shape<H, L>::kBChunks * kChunk];   // [delta_1 | ... | delta_L | gy]
  unsigned char w1[4 * H * 16];                      // B operands of the forward
  unsigned char wl[(L > 1 ? L - 1 : 1) * 2 * H * H];
  unsigned char w1t[4 * H * 16];                     // B[n = k][kk = i] = W_1[i][k], N = 32
  unsigned char wlt[(L > 1 ? L - 1 : 1) * 2 * H * H];// B[n = i][k = j] = W[j][i]
  float woutf[3 * H];
  unsigned long long bar;
  uint32_t tmem_base;
  uint32_t failed;
};

// kGather: only the Gaussians whose bit is set in a.flags are worked on and written.  Every CTA takes one contiguous
// run of flag words, reads it 32 words at a time (thread t looks at byte t % 4 of word t / 4, an exclusive scan over the
// CTA gives its place in a queue in shared memory, it writes the indices of its set bits there: index order, the same
// from run to run) and runs a tile whenever 128 indices are queued, and once more for what is left.
constexpr int kGatherWords = tc::kTile / 4;               // flag words per round
constexpr int kGatherQueue = 2 * 32 * kGatherWords;       // a power of two above 32 kGatherWords + 127

template <int H, int L, bool kGather>
__global__ void __launch_bounds__(tc::kTile, H == 16 ? 4 : 2) k_variant_bwd_tc(AppearanceArgs a, int nfeat) {
  using S_t = SmemBwd<H, L>;
  using Sh = Shape<H, L>;
  using D = VarDims<H, L>;
  extern __shared__ __align__(128) unsigned char vtc_smem[];
  S_t &S = *reinterpret_cast<S_t *>(vtc_smem);
  const int tid = threadIdx.x, warp = tid >> 5;
  stage_weights<H, L>(a.weights, S.w1, S.wl, S.woutf, S.w1t, S.wlt, tid);
  const uint32_t bar = tc::smem_addr(&S.bar);
  if (tid == 0) {
    tc::barrier_init(bar);
    tc::fence_barrier_init();
    S.failed = 0u;
  }
  if (warp == 0) tc::tmem_alloc(&S.tmem_base, (uint32_t)Sh::kColsAlloc);
  tc::fence_generic_writes();
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t *>(&S.tmem_base);
  const uint32_t my_lane = tmem + ((uint32_t)(warp * 32) << 16);
  const uint32_t A4 = tc::smem_addr(S.a) >> 4, B4 = tc::smem_addr(S.b) >> 4;
  const uint32_t W14 = tc::smem_addr(S.w1) >> 4, WL4 = tc::smem_addr(S.wl) >> 4, W1T4 = tc::smem_addr(S.w1t) >> 4, WLT4 = tc::smem_addr(S.wlt) >> 4;
  constexpr uint32_t kDW = Sh::kChainCols;
  uint32_t phase = 0;
  bool first_tile = true;
  auto run_phase = [&](auto issue) {
    tc::fence_generic_writes();
    tc::fence_before_sync();
    __syncthreads();
    if (tid == 0 && !*reinterpret_cast<volatile uint32_t *>(&S.failed)) {
      tc::fence_after_sync();
      issue();
      tc::commit(bar);
    }
    if (!*reinterpret_cast<volatile uint32_t *>(&S.failed)) {
      if (!tc::wait_phase(bar, phase & 1u)) {
        S.failed = 1u;
        if (a.timeout) atomicExch(a.timeout, 1ull);
      }
    }
    ++phase;
    tc::fence_after_sync();
  };
  // one tile: thread t works on Gaussian i (exists: it has one)
  auto do_tile = [&](const int64_t i, const bool exists) {
    const bool in = exists && (!a.mask || __ldg(a.mask + i) != 0u);
    float d[3] = {0.f, 0.f, 1.f}, base[3] = {0.f, 0.f, 0.f}, gcol[3] = {0.f, 0.f, 0.f};
    float xs[16];                        // inputs 16..31 ((sin, cos) pairs or raw features), needed again for dL/df
    {
      float x[32];
      if (in) {
#pragma unroll
        for (int c = 0; c < 3; ++c) base[c] = __ldg(a.base_color + 3 * i + c);
        if (kGather && a.g2d) {          // inside the step: the direction as the forward took it, dL/dcolor where the blend left it
          const float vx = __ldg(a.means + 3 * i) - a.oc[0], vy = __ldg(a.means + 3 * i + 1) - a.oc[1], vz = __ldg(a.means + 3 * i + 2) - a.oc[2];
          const float vi = rsqrtf(vx * vx + vy * vy + vz * vz);
          d[0] = vx * vi; d[1] = vy * vi; d[2] = vz * vi;
          const float4 ga = __ldg(reinterpret_cast<const float4 *>(a.g2d) + 3 * i);
          gcol[0] = ga.x; gcol[1] = ga.y; gcol[2] = ga.z;
        } else {
#pragma unroll
          for (int c = 0; c < 3; ++c) { d[c] = __ldg(a.dirs + 3 * i + c); gcol[c] = __ldg(a.g_color + 3 * i + c); }
        }
        inputs(a, i, nfeat, d, x);
      } else {
#pragma unroll
        for (int k = 0; k < 32; ++k) x[k] = 0.f;
      }
#pragma unroll
      for (int k = 0; k < 16; ++k) xs[k] = x[16 + k];
      store_row<32>(S.a, tid, x);
    }
    // ---- forward: h_l = relu(h_(l-1) W_l^T), every layer's rows kept
    uint32_t m[L];                       // relu'(h_l) as bit masks
    float h[H];
    run_phase([&] { tc::rows_times<2, 2, H, 4u * kChunk>(tmem, A4, W14, tc::idesc(128, H)); });
#pragma unroll
    for (int l = 1; l <= L; ++l) {
      load_row<H>(my_lane, h);
      m[l - 1] = 0u;
#pragma unroll
      for (int k = 0; k < H; ++k) { m[l - 1] |= (h[k] > 0.f ? 1u : 0u) << k; h[k] = fmaxf(h[k], 0.f); }
      store_row<H>(S.a + Sh::a_start(l) * kChunk, tid, h);
      if (l < L)
        run_phase([&] {
          tc::rows_times<2, Sh::kHS, H, Sh::kHC * kChunk>(tmem, A4 + (uint32_t)(Sh::a_start(l) * kChunk >> 4), WL4 + (uint32_t)((l - 1) * 2 * H * H >> 4), tc::idesc(128, H));
        });
    }
    float gp[3], gy[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    {
      float y[3];
      output_layer<H>(S.woutf, h, y);
#pragma unroll
      for (int c = 0; c < 3; ++c) {
        const float A = tanh_fast(y[c]);
        gp[c] = in ? color_act_grad_z(a.act, base[c] + 0.5f + A) * gcol[c] : 0.f;
        gy[c] = gp[c] * (1.f - A * A);
      }
    }
    tc::store_chunk<true>(S.b + Sh::b_start(L) * kChunk, S.b + (Sh::b_start(L) + 1) * kChunk, (uint32_t)tid * 16u, gy);
    // ---- delta_L = (gy W_out) relu'(h_L), then delta_l = (delta_(l+1) W_(l+1)) relu'(h_l)
#pragma unroll
    for (int q = 0; q < H / 4; ++q) {
      const float4 r0 = *reinterpret_cast<const float4 *>(S.woutf + 4 * q), r1 = *reinterpret_cast<const float4 *>(S.woutf + H + 4 * q),
                   r2 = *reinterpret_cast<const float4 *>(S.woutf + 2 * H + 4 * q);
      h[4 * q] = fmaf(gy[0], r0.x, fmaf(gy[1], r1.x, gy[2] * r2.x));
      h[4 * q + 1] = fmaf(gy[0], r0.y, fmaf(gy[1], r1.y, gy[2] * r2.y));
      h[4 * q + 2] = fmaf(gy[0], r0.z, fmaf(gy[1], r1.z, gy[2] * r2.z));
      h[4 * q + 3] = fmaf(gy[0], r0.w, fmaf(gy[1], r1.w, gy[2] * r2.w));
    }
#pragma unroll
    for (int l = L; l >= 1; --l) {       // h = delta_l before its mask
#pragma unroll
      for (int k = 0; k < H; ++k) h[k] = (m[l - 1] >> k) & 1u ? h[k] : 0.f;
      store_row<H>(S.b + Sh::b_start(l - 1) * kChunk, tid, h);
      if (l > 1) {
        run_phase([&] {
          tc::rows_times<2, Sh::kHS, H, Sh::kHC * kChunk>(tmem, B4 + (uint32_t)(Sh::b_start(l - 1) * kChunk >> 4), WLT4 + (uint32_t)((l - 2) * 2 * H * H >> 4), tc::idesc(128, H));
        });
        load_row<H>(my_lane, h);
      }
    }
    // ---- gx = delta_1 W_1, and the weight gradients of the tile: K runs over its 128 rows, 16 per MMA
    const bool fresh = first_tile;
    run_phase([&] {
      if (Sh::kSplitGx) tc::rows_times<2, Sh::kHS, 32, Sh::kHC * kChunk>(tmem, B4, W1T4, tc::idesc(128, 16));   // rows 0..15 of W_1^T
      else tc::rows_times<2, Sh::kHS, 32, Sh::kHC * kChunk>(tmem, B4, W1T4, tc::idesc(128, 32));
#pragma unroll
      for (int b = 0; b < Sh::kBlocks; ++b)
#pragma unroll
        for (int ks = 0; ks < tc::kTile / 16; ++ks)
          tc::mma(tmem + kDW + (uint32_t)Sh::dw_col(b), tc::desc_at<128u, kChunk>(A4, (uint32_t)b * 16u * kChunk + (uint32_t)ks * 256u),
                  tc::desc_at<128u, kChunk>(B4, (uint32_t)Sh::n_start(b) * kChunk + (uint32_t)ks * 256u), (fresh && ks == 0) ? 0u : 1u,
                  tc::idesc(128, Sh::n_cols(b), true, true));
    });
    first_tile = false;
    float gx[32];
    if (Sh::kSplitGx) {
      load_row<16>(my_lane, gx);
      run_phase([&] { tc::rows_times<2, Sh::kHS, 32, Sh::kHC * kChunk>(tmem, B4, W1T4 + (16u * 16u >> 4), tc::idesc(128, 16)); });   // rows 16..31
      load_row<16>(my_lane, gx + 16);
    } else {
      load_row<32>(my_lane, gx);
    }
    if (exists) {
      a.g_base[3 * i] = gp[0]; a.g_base[3 * i + 1] = gp[1]; a.g_base[3 * i + 2] = gp[2];
      if (nfeat == 8) {
        float gf[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) gf[j] = gx[16 + 2 * j] * xs[2 * j + 1] - gx[17 + 2 * j] * xs[2 * j];
        float4 *dst = reinterpret_cast<float4 *>(a.g_features) + 2 * i;
        dst[0] = make_float4(gf[0], gf[1], gf[2], gf[3]); dst[1] = make_float4(gf[4], gf[5], gf[6], gf[7]);
      } else {
        float4 *dst = reinterpret_cast<float4 *>(a.g_features) + 4 * i;
#pragma unroll
        for (int q = 0; q < 4; ++q) dst[q] = make_float4(gx[16 + 4 * q], gx[17 + 4 * q], gx[18 + 4 * q], gx[19 + 4 * q]);
      }
      const int na = (a.deg + 1) * (a.deg + 1);
      float ax = 0.f, ay = 0.f, az = 0.f;
#pragma unroll
      for (int k = 1; k < 16; ++k)
        if (k < na) sh_grad_acc(k, d[0], d[1], d[2], gx[k], ax, ay, az);
      a.g_dirs[3 * i] = ax; a.g_dirs[3 * i + 1] = ay; a.g_dirs[3 * i + 2] = az;
    }
  };
  if constexpr (!kGather) {
    const int64_t ntiles = (a.n + tc::kTile - 1) / tc::kTile;
    for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
      const int64_t i = tile * tc::kTile + tid;
      do_tile(i, i < a.n);
    }
  } else {
    __shared__ uint32_t s_queue[kGatherQueue];
    __shared__ int s_warp_count[tc::kTile / 32];
    constexpr int kMask = kGatherQueue - 1;
    const int lane = tid & 31;
    int q_head = 0, q_count = 0;         // the same in every thread
    const int64_t nwords = (a.n + 31) / 32, per_cta = (nwords + gridDim.x - 1) / gridDim.x;
    const int64_t w_begin = min(nwords, (int64_t)blockIdx.x * per_cta), w_end = min(nwords, w_begin + per_cta);
    for (int64_t w0 = w_begin; w0 < w_end; w0 += kGatherWords) {
      const int64_t w = w0 + (tid >> 2);
      const uint32_t byte = w < w_end ? (__ldg(a.flags + w) >> (8 * (tid & 3))) & 255u : 0u;
      const int cnt = __popc(byte);
      int incl = cnt;
#pragma unroll
      for (int sft = 1; sft < 32; sft <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, sft);
        if (lane >= sft) incl += t;
      }
      if (lane == 31) s_warp_count[warp] = incl;
      __syncthreads();
      int offset = incl - cnt, total = 0;
#pragma unroll
      for (int ww = 0; ww < tc::kTile / 32; ++ww) { const int c = s_warp_count[ww]; offset += ww < warp ? c : 0; total += c; }
      uint32_t bits = byte;
      const uint32_t row0 = (uint32_t)(w * 32 + 8 * (tid & 3));
      for (int slot = q_head + q_count + offset; bits; ++slot) {
        const int b = __ffs(bits) - 1;
        bits &= bits - 1u;
        s_queue[slot & kMask] = row0 + (uint32_t)b;
      }
      __syncthreads();
      q_count += total;
      while (q_count >= tc::kTile) {
        do_tile((int64_t)s_queue[(q_head + tid) & kMask], true);
        q_head = (q_head + tc::kTile) & kMask;
        q_count -= tc::kTile;
        __syncthreads();
      }
    }
    if (q_count > 0) do_tile(tid < q_count ? (int64_t)s_queue[(q_head + tid) & kMask] : 0, tid < q_count);
  }
  // ---- this CTA's partial of the weight gradient.  In block b, thread t holds the row of column 128 b + t of
  // [X | h_1 | ...]; of that row it reads its partner's columns and adds the high- and low-half columns.
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  float *tmp = reinterpret_cast<float *>(S.a);            // [8 kAChunks][H]
#pragma unroll
  for (int b = 0; b < Sh::kBlocks; ++b) {
    const int e0 = 128 * b + 32 * warp;                   // first row of this warp in the block: one buffer per warp
    const int j = e0 < 64 ? 0 : 1 + (e0 - 64) / (2 * H);
    if (j <= L) {
      const uint32_t col = kDW + (uint32_t)Sh::dw_col(b) + 8u * (uint32_t)(Sh::b_start(j) - Sh::n_start(b));
      float v[H];
      if (j < L) {
        float lo[H];
        load_row<H>(my_lane + col, v);
        load_row<H>(my_lane + col + (uint32_t)H, lo);
#pragma unroll
        for (int k = 0; k < H; ++k) v[k] += lo[k];
      } else {
        float g[16];
        tc::load16(my_lane + col, g);
#pragma unroll
        for (int k = 0; k < H; ++k) v[k] = k < 8 ? g[k] + g[8 + k] : 0.f;
      }
#pragma unroll
      for (int k = 0; k < H; ++k) tmp[(128 * b + tid) * H + k] = first_tile ? 0.f : v[k];
    }
  }
  __syncthreads();
  float *out = a.w_partials + (size_t)blockIdx.x * D::kNumW;
  for (int idx = tid; idx < H * 32; idx += tc::kTile) {     // dW_1[i][k]: rows k (high) and 32 + k (low) of X, column i
    const int i = idx >> 5, k = idx & 31;
    out[idx] = tmp[k * H + i] + tmp[(32 + k) * H + i];
  }
  for (int l = 1; l <= L; ++l) {                            // rows of h_l: dW_(l+1)[o][i] (or dW_out[c][i]) = rows i, column o
    const int e = 64 + (l - 1) * 2 * H, nout = l < L ? H : 3;
    for (int idx = tid; idx < nout * H; idx += tc::kTile) {
      const int o = idx / H, i2 = idx % H;
      out[D::off(l) + idx] = tmp[(e + i2) * H + o] + tmp[(e + H + i2) * H + o];
    }
  }
  __syncthreads();
  if (warp == 0) tc::tmem_free(tmem, (uint32_t)Sh::kColsAlloc);
}

}  // namespace vtc
