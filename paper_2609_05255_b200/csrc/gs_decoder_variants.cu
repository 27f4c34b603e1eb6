// The decoder variants of the paper's architecture table (App. D): 1 to 3 hidden layers of 16 or 32
// neurons, 8 frequency-encoded or 16 raw features, evaluated in the separate-pass path (the path the paper
// calls "without fusion").  Two engines: the tcgen05 kernels of gs_variants_tc.cuh (the default), and the
// kernels of this file, plain fp32 FMAs with the weights in shared memory, one thread per Gaussian (the second
// engine, and the path of degree 0, where nothing is decoded).  In the fp32 backward the weight gradient - a
// contraction over Gaussians - is taken per warp: it stages the inputs and output gradients of its 32 Gaussians in shared memory, every lane owns every 32nd
// weight of the layer and sums its 32 products, and the per-warp sums (kept in shared memory, one owner per
// element, so no atomics) leave as per-block partials that a last kernel adds up in a fixed order.
#include <cuda_fp16.h>

#include "gs_device.cuh"

namespace gs {
namespace {

constexpr int kVarBlock = 128;
constexpr int kVarWarps = kVarBlock / 32;
constexpr int kVarPartialBlocks = 592;   // most persistent CTAs of the backward (rows of the partial buffer)

template <int H, int L> struct VarDims {
  static constexpr int kNumW = 32 * H + (L - 1) * H * H + 3 * H;
  __host__ __device__ static constexpr int off(int l) { return l == 0 ? 0 : 32 * H + (l - 1) * H * H; }   // matrix l of 0..L
};

__device__ __forceinline__ void variant_inputs(const AppearanceArgs &a, int64_t i, int nfeat, const float d[3], float x[32]) {
  float Y[16];
  sh_basis(d[0], d[1], d[2], Y);
  const int na = (a.deg + 1) * (a.deg + 1);
#pragma unroll
  for (int k = 0; k < 16; ++k) x[k] = k < na ? Y[k] : 0.f;
  if (nfeat == 8) {
    const uint4 raw = __ldg(reinterpret_cast<const uint4 *>(a.features) + i);
    const __half2 *h = reinterpret_cast<const __half2 *>(&raw);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float2 f = __half22float2(h[j]);
      sincosf(f.x, &x[16 + 4 * j], &x[17 + 4 * j]);
      sincosf(f.y, &x[18 + 4 * j], &x[19 + 4 * j]);
    }
  } else {
    const uint4 r0 = __ldg(reinterpret_cast<const uint4 *>(a.features) + 2 * i), r1 = __ldg(reinterpret_cast<const uint4 *>(a.features) + 2 * i + 1);
    const __half2 *h0 = reinterpret_cast<const __half2 *>(&r0), *h1 = reinterpret_cast<const __half2 *>(&r1);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float2 f = __half22float2(h0[j]), g = __half22float2(h1[j]);
      x[16 + 2 * j] = f.x; x[17 + 2 * j] = f.y; x[24 + 2 * j] = g.x; x[25 + 2 * j] = g.y;
    }
  }
}

#include "gs_variants_tc.cuh"

// y[o] = sum_i W[o][i] in[i]; the weights are read as shared-memory broadcasts.
template <int NOUT, int NIN>
__device__ __forceinline__ void matvec(const float *W, const float in[NIN], float out[NOUT]) {
#pragma unroll
  for (int o = 0; o < NOUT; ++o) {
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < NIN; i += 4) {
      const float4 w = *reinterpret_cast<const float4 *>(W + o * NIN + i);
      acc = fmaf(w.x, in[i], acc); acc = fmaf(w.y, in[i + 1], acc); acc = fmaf(w.z, in[i + 2], acc); acc = fmaf(w.w, in[i + 3], acc);
    }
    out[o] = acc;
  }
}
// gin[i] = sum_o W[o][i] gout[o]
template <int NOUT, int NIN>
__device__ __forceinline__ void matvec_t(const float *W, const float gout[NOUT], float gin[NIN]) {
#pragma unroll
  for (int i = 0; i < NIN; ++i) gin[i] = 0.f;
#pragma unroll
  for (int o = 0; o < NOUT; ++o) {
#pragma unroll
    for (int i = 0; i < NIN; i += 4) {
      const float4 w = *reinterpret_cast<const float4 *>(W + o * NIN + i);
      gin[i] = fmaf(w.x, gout[o], gin[i]); gin[i + 1] = fmaf(w.y, gout[o], gin[i + 1]);
      gin[i + 2] = fmaf(w.z, gout[o], gin[i + 2]); gin[i + 3] = fmaf(w.w, gout[o], gin[i + 3]);
    }
  }
}

template <int H, int L>
struct VarState { float x[32], h[L][H], A[3]; };

template <int H, int L>
__device__ __forceinline__ void variant_forward(const float *sW, VarState<H, L> &s) {
  matvec<H, 32>(sW, s.x, s.h[0]);
#pragma unroll
  for (int o = 0; o < H; ++o) s.h[0][o] = fmaxf(s.h[0][o], 0.f);
#pragma unroll
  for (int l = 1; l < L; ++l) {
    matvec<H, H>(sW + VarDims<H, L>::off(l), s.h[l - 1], s.h[l]);
#pragma unroll
    for (int o = 0; o < H; ++o) s.h[l][o] = fmaxf(s.h[l][o], 0.f);
  }
  float y[3];
  matvec<3, H>(sW + VarDims<H, L>::off(L), s.h[L - 1], y);
#pragma unroll
  for (int c = 0; c < 3; ++c) s.A[c] = tanhf(y[c]);
}

template <int H, int L>
__global__ void __launch_bounds__(kVarBlock) k_variant_fwd(AppearanceArgs a, int nfeat) {
  extern __shared__ __align__(16) float sW[];
  for (int k = threadIdx.x; k < VarDims<H, L>::kNumW; k += kVarBlock) sW[k] = __half2float(a.weights[k]);
  __syncthreads();
  const int64_t i = (int64_t)blockIdx.x * kVarBlock + threadIdx.x;
  if (i >= a.n || (a.mask && __ldg(a.mask + i) == 0u)) return;   // masked-out Gaussians are skipped
  float d[3], base[3];
  d[0] = __ldg(a.dirs + 3 * i); d[1] = __ldg(a.dirs + 3 * i + 1); d[2] = __ldg(a.dirs + 3 * i + 2);
  base[0] = __ldg(a.base_color + 3 * i); base[1] = __ldg(a.base_color + 3 * i + 1); base[2] = __ldg(a.base_color + 3 * i + 2);
  VarState<H, L> s;
  s.A[0] = s.A[1] = s.A[2] = 0.f;
  if (a.deg > 0) {
    variant_inputs(a, i, nfeat, d, s.x);
    variant_forward<H, L>(sW, s);
  }
#pragma unroll
  for (int c = 0; c < 3; ++c) a.color[3 * i + c] = color_act_z(a.act, base[c] + 0.5f + s.A[c]);
}

// Weight gradient of one layer for the warp's 32 Gaussians: sX [32][NIN] inputs, sG [32][NOUT] output gradients
// (rows of Gaussians without one are zero).  A lane owns one input column and four output rows at a time, so one
// load of the input and one 16-byte load of the gradients feed four FMAs; the sums of every element are taken in
// Gaussian order by its one owner.
template <int NOUT, int NIN>
__device__ __forceinline__ void warp_weight_grad(const float *sX, const float *sG, float *sDW, int lane) {
  if (NOUT % 4 != 0) {   // the three output rows
    for (int w = lane; w < NOUT * NIN; w += 32) {
      const int o = w / NIN, i = w % NIN;
      float acc = sDW[w];
#pragma unroll 8
      for (int g = 0; g < 32; ++g) acc = fmaf(sG[g * NOUT + o], sX[g * NIN + i], acc);
      sDW[w] = acc;
    }
    return;
  }
  constexpr int kGroups = 32 / NIN;   // lanes per column
  const int i = lane % NIN, og = lane / NIN;
  for (int c = og; c < NOUT / 4; c += kGroups) {
    float acc[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) acc[r] = sDW[(4 * c + r) * NIN + i];
#pragma unroll 8
    for (int g = 0; g < 32; ++g) {
      const float x = sX[g * NIN + i];
      const float4 gg = *reinterpret_cast<const float4 *>(sG + g * NOUT + 4 * c);
      acc[0] = fmaf(gg.x, x, acc[0]); acc[1] = fmaf(gg.y, x, acc[1]);
      acc[2] = fmaf(gg.z, x, acc[2]); acc[3] = fmaf(gg.w, x, acc[3]);
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) sDW[(4 * c + r) * NIN + i] = acc[r];
  }
}

template <int H, int L>
__global__ void __launch_bounds__(kVarBlock) k_variant_bwd(AppearanceArgs a, int nfeat) {
  using D = VarDims<H, L>;
  extern __shared__ __align__(16) float smem[];
  float *sW = smem;                                             // [kNumW]
  float *sDWall = sW + D::kNumW;                                // [kVarWarps][kNumW]
  float *sStage = sDWall + kVarWarps * D::kNumW;                // [kVarWarps][32 x 32 + 32 x 32]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int k = tid; k < D::kNumW; k += kVarBlock) sW[k] = __half2float(a.weights[k]);
  for (int k = tid; k < kVarWarps * D::kNumW; k += kVarBlock) sDWall[k] = 0.f;
  __syncthreads();
  float *sDW = sDWall + warp * D::kNumW;
  float *sX = sStage + warp * 2048, *sG = sX + 1024;
  const int64_t nchunks = (a.n + kVarBlock - 1) / kVarBlock;
  for (int64_t chunk = blockIdx.x; chunk < nchunks; chunk += gridDim.x) {
    const int64_t i = chunk * kVarBlock + tid;
    const bool exists = i < a.n;
    const bool in = exists && (!a.mask || __ldg(a.mask + i) != 0u);   // masked out: zero gradient rows
    float d[3] = {0.f, 0.f, 1.f}, base[3] = {0.f, 0.f, 0.f}, gcol[3] = {0.f, 0.f, 0.f};
    if (in) {
#pragma unroll
      for (int c = 0; c < 3; ++c) { d[c] = __ldg(a.dirs + 3 * i + c); base[c] = __ldg(a.base_color + 3 * i + c); gcol[c] = __ldg(a.g_color + 3 * i + c); }
    }
    float gp[3], gx[32];
#pragma unroll
    for (int k = 0; k < 32; ++k) gx[k] = 0.f;
    if (a.deg == 0) {
#pragma unroll
      for (int c = 0; c < 3; ++c) gp[c] = color_act_grad_z(a.act, base[c] + 0.5f) * gcol[c];
    } else {
      VarState<H, L> s;
      if (in) {
        variant_inputs(a, i, nfeat, d, s.x);
      } else {
#pragma unroll
        for (int k = 0; k < 32; ++k) s.x[k] = 0.f;
      }
      variant_forward<H, L>(sW, s);
      float g_hi[H > 3 ? H : 3];                                // gradient at the outputs of the current matrix
#pragma unroll
      for (int c = 0; c < 3; ++c) {
        gp[c] = in ? color_act_grad_z(a.act, base[c] + 0.5f + s.A[c]) * gcol[c] : 0.f;
        g_hi[c] = gp[c] * (1.f - s.A[c] * s.A[c]);
      }
      // ---- output matrix: [3][H]
      {
        __syncwarp();
#pragma unroll
        for (int k = 0; k < H; ++k) sX[lane * H + k] = s.h[L - 1][k];
#pragma unroll
        for (int c = 0; c < 3; ++c) sG[lane * 3 + c] = g_hi[c];
        __syncwarp();
        warp_weight_grad<3, H>(sX, sG, sDW + D::off(L), lane);
        float g_lo[H];
        matvec_t<3, H>(sW + D::off(L), g_hi, g_lo);
#pragma unroll
        for (int k = 0; k < H; ++k) g_hi[k] = s.h[L - 1][k] > 0.f ? g_lo[k] : 0.f;
      }
      // ---- hidden matrices L-1 .. 1: [H][H]
#pragma unroll
      for (int l = L - 1; l >= 1; --l) {
        __syncwarp();
#pragma unroll
        for (int k = 0; k < H; ++k) { sX[lane * H + k] = s.h[l - 1][k]; sG[lane * H + k] = g_hi[k]; }
        __syncwarp();
        warp_weight_grad<H, H>(sX, sG, sDW + D::off(l), lane);
        float g_lo[H];
        matvec_t<H, H>(sW + D::off(l), g_hi, g_lo);
#pragma unroll
        for (int k = 0; k < H; ++k) g_hi[k] = s.h[l - 1][k] > 0.f ? g_lo[k] : 0.f;
      }
      // ---- first matrix: [H][32]
      __syncwarp();
#pragma unroll
      for (int k = 0; k < 32; ++k) sX[lane * 32 + k] = s.x[k];
#pragma unroll
      for (int k = 0; k < H; ++k) sG[lane * H + k] = g_hi[k];
      __syncwarp();
      warp_weight_grad<H, 32>(sX, sG, sDW, lane);
      matvec_t<H, 32>(sW, g_hi, gx);
    }
    if (exists) {
      a.g_base[3 * i] = gp[0]; a.g_base[3 * i + 1] = gp[1]; a.g_base[3 * i + 2] = gp[2];
      // features
      if (nfeat == 8) {
        float gf[8];
        if (a.deg > 0 && in) {
          float x[32];
          variant_inputs(a, i, nfeat, d, x);
#pragma unroll
          for (int j = 0; j < 8; ++j) gf[j] = gx[16 + 2 * j] * x[17 + 2 * j] - gx[17 + 2 * j] * x[16 + 2 * j];
        } else {
#pragma unroll
          for (int j = 0; j < 8; ++j) gf[j] = 0.f;
        }
        float4 *dst = reinterpret_cast<float4 *>(a.g_features) + 2 * i;
        dst[0] = make_float4(gf[0], gf[1], gf[2], gf[3]); dst[1] = make_float4(gf[4], gf[5], gf[6], gf[7]);
      } else {
        float4 *dst = reinterpret_cast<float4 *>(a.g_features) + 4 * i;
#pragma unroll
        for (int q = 0; q < 4; ++q) dst[q] = make_float4(gx[16 + 4 * q], gx[17 + 4 * q], gx[18 + 4 * q], gx[19 + 4 * q]);
      }
      // direction: chain through the SH basis
      const int na = (a.deg + 1) * (a.deg + 1);
      float ax = 0.f, ay = 0.f, az = 0.f;
#pragma unroll
      for (int k = 1; k < 16; ++k)
        if (k < na) sh_grad_acc(k, d[0], d[1], d[2], gx[k], ax, ay, az);
      a.g_dirs[3 * i] = ax; a.g_dirs[3 * i + 1] = ay; a.g_dirs[3 * i + 2] = az;
    }
  }
  __syncthreads();
  float *partial = a.w_partials + (size_t)blockIdx.x * D::kNumW;
  for (int k = tid; k < D::kNumW; k += kVarBlock) {
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < kVarWarps; ++w) t += sDWall[w * D::kNumW + k];
    partial[k] = t;
  }
}

// Deterministic sum of the per-block partials: 32 weights per CTA, the rows shared out over sixteen groups of threads
// (each sums every sixteenth row, in order, four loads in flight), the sixteen sums added in a fixed order.
constexpr int kVarReduceGroups = 16;
__global__ void __launch_bounds__(32 * kVarReduceGroups) k_variant_wreduce(const float *__restrict__ partials, int nblocks, int nw,
                                                                           float *__restrict__ out) {
  __shared__ float s_part[kVarReduceGroups][32];
  const int k = blockIdx.x * 32 + threadIdx.x, grp = threadIdx.y;
  float s = 0.f;
  if (k < nw) {
    int b = grp;
    for (; b + 3 * kVarReduceGroups < nblocks; b += 4 * kVarReduceGroups) {
      const float p0 = partials[(size_t)b * nw + k], p1 = partials[(size_t)(b + kVarReduceGroups) * nw + k],
                  p2 = partials[(size_t)(b + 2 * kVarReduceGroups) * nw + k], p3 = partials[(size_t)(b + 3 * kVarReduceGroups) * nw + k];
      s += p0; s += p1; s += p2; s += p3;
    }
    for (; b < nblocks; b += kVarReduceGroups) s += partials[(size_t)b * nw + k];
  }
  s_part[grp][threadIdx.x] = s;
  __syncthreads();
  if (grp == 0 && k < nw) {
    float t = 0.f;
#pragma unroll
    for (int q = 0; q < kVarReduceGroups; ++q) t += s_part[q][threadIdx.x];
    out[k] = t;
  }
}
inline void launch_variant_wreduce(const float *partials, int nblocks, int nw, float *out, cudaStream_t st) {
  k_variant_wreduce<<<(nw + 31) / 32, dim3(32, kVarReduceGroups), 0, st>>>(partials, nblocks, nw, out);
}

template <class K>
void opt_in(K kernel, size_t bytes) { cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes); }

template <int H, int L>
int run_fwd(const AppearanceArgs &a, int nfeat, cudaStream_t st) {
  const size_t smem = sizeof(float) * VarDims<H, L>::kNumW;
  opt_in(k_variant_fwd<H, L>, smem);
  k_variant_fwd<H, L><<<(unsigned)((a.n + kVarBlock - 1) / kVarBlock), kVarBlock, smem, st>>>(a, nfeat);
  return 1;
}
template <int H, int L>
int run_bwd(const AppearanceArgs &a, int nfeat, cudaStream_t st) {
  using D = VarDims<H, L>;
  const size_t smem = sizeof(float) * ((1 + kVarWarps) * D::kNumW + kVarWarps * 2048);
  opt_in(k_variant_bwd<H, L>, smem);
  const int64_t chunks = (a.n + kVarBlock - 1) / kVarBlock;
  // one full wave: as many CTAs as are resident at once
  int per_sm = 0, sms = 0, dev = 0, wave = kVarPartialBlocks;
  if (cudaGetDevice(&dev) == cudaSuccess &&
      cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_variant_bwd<H, L>, kVarBlock, smem) == cudaSuccess &&
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && per_sm > 0 && sms > 0)
    wave = per_sm * sms < kVarPartialBlocks ? per_sm * sms : kVarPartialBlocks;
  const int blocks = (int)(chunks < wave ? chunks : wave);
  k_variant_bwd<H, L><<<blocks, kVarBlock, smem, st>>>(a, nfeat);
  launch_variant_wreduce(a.w_partials, blocks, D::kNumW, a.g_weights, st);
  return 2;
}

int sm_count() {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) sms = 148;
  return sms;
}

// The tcgen05 kernels: persistent grids of one full wave.  The occupancy query does not see tensor memory, so the
// resident CTAs per SM are taken from the three budgets directly: 512 columns of tensor memory, 228 KB of shared
// memory (1 KB per CTA is the system's), 64 K registers.
template <int H, int L>
int run_fwd_tc(const AppearanceArgs &a, int nfeat, cudaStream_t st) {
  const size_t smem = sizeof(vtc::SmemFwd<H, L>);
  opt_in(vtc::k_variant_fwd_tc<H, L>, smem);
  const int64_t tiles = (a.n + tc::kTile - 1) / tc::kTile;
  const int64_t wave = (int64_t)(H == 16 ? 8 : 7) * sm_count();   // 59 and 71 registers per thread
  vtc::k_variant_fwd_tc<H, L><<<(unsigned)(tiles < wave ? tiles : wave), tc::kTile, smem, st>>>(a, nfeat);
  return 1;
}
template <int H, int L>
int run_bwd_tc(const AppearanceArgs &a, int nfeat, cudaStream_t st) {
  using D = VarDims<H, L>;
  const size_t smem = sizeof(vtc::SmemBwd<H, L>);
  const bool gather = a.flags != nullptr;
  opt_in(vtc::k_variant_bwd_tc<H, L, false>, smem);
  opt_in(vtc::k_variant_bwd_tc<H, L, true>, smem);
  int per_sm = 512 / vtc::Shape<H, L>::kColsAlloc;
  const int by_smem = (int)((228 * 1024) / (smem + 1024 + (gather ? sizeof(uint32_t) * vtc::kGatherQueue + 64 : 0)));
  if (by_smem < per_sm) per_sm = by_smem;
  if (per_sm > (H == 16 ? 4 : 2)) per_sm = H == 16 ? 4 : 2;   // registers: the launch bounds of the kernel
  if (per_sm < 1) per_sm = 1;
  const int64_t tiles = (a.n + tc::kTile - 1) / tc::kTile;
  int64_t wave = (int64_t)per_sm * sm_count();
  if (wave > kVarPartialBlocks) wave = kVarPartialBlocks;
  const int blocks = (int)(tiles < wave ? tiles : wave);
  if (gather) vtc::k_variant_bwd_tc<H, L, true><<<blocks, tc::kTile, smem, st>>>(a, nfeat);
  else vtc::k_variant_bwd_tc<H, L, false><<<blocks, tc::kTile, smem, st>>>(a, nfeat);
  launch_variant_wreduce(a.w_partials, blocks, D::kNumW, a.g_weights, st);
  return 2;
}

}  // namespace

int variant_num_weights(int hidden, int layers) { return 32 * hidden + (layers - 1) * hidden * hidden + 3 * hidden; }
size_t variant_partials_floats() { return (size_t)kVarPartialBlocks * VarDims<32, 3>::kNumW; }

#define GS_VARIANT_DISPATCH(FN)                                        \
  if (hidden == 16 && layers == 1) return FN<16, 1>(a, nfeat, st);      \
  if (hidden == 16 && layers == 2) return FN<16, 2>(a, nfeat, st);      \
  if (hidden == 16 && layers == 3) return FN<16, 3>(a, nfeat, st);      \
  if (hidden == 32 && layers == 1) return FN<32, 1>(a, nfeat, st);      \
  if (hidden == 32 && layers == 2) return FN<32, 2>(a, nfeat, st);      \
  if (hidden == 32 && layers == 3) return FN<32, 3>(a, nfeat, st);      \
  return -1;

int launch_variant_fwd(int hidden, int layers, int nfeat, const AppearanceArgs &a, cudaStream_t st) {
  if (a.n == 0) return 0;
  if (a.engine != GS_ENGINE_WARP_MMA && a.deg > 0) { GS_VARIANT_DISPATCH(run_fwd_tc) }
  GS_VARIANT_DISPATCH(run_fwd)
}
int launch_variant_bwd(int hidden, int layers, int nfeat, const AppearanceArgs &a, cudaStream_t st) {
  if (a.n == 0) {
    cudaMemsetAsync(a.g_weights, 0, sizeof(float) * variant_num_weights(hidden, layers), st);
    return 0;
  }
  if (a.engine != GS_ENGINE_WARP_MMA && a.deg > 0) { GS_VARIANT_DISPATCH(run_bwd_tc) }
  GS_VARIANT_DISPATCH(run_bwd)
}

}  // namespace gs
