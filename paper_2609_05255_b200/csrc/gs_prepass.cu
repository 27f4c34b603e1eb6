// Viewer-side evaluation of the neural appearance model (App. C.3, "Neural"), as CUDA kernels instead
// of fragment shaders.  Export: the 17 view-independent columns of the first layer (16 encoded
// features + the constant degree-0 input) are folded into 16 half-precision pre-activations per
// Gaussian.  Per frame: the 15 direction-dependent columns (padded to 16) and the two later layers,
// 560 multiply-accumulates per Gaussian, in half precision on tensor cores with fp32 accumulation,
// and one 8-bit RGBA texel per Gaussian as the result.
#include <cuda_fp16.h>

#include "gs_device.cuh"
#include "gs_mlp_mma.cuh"

namespace gs {
namespace {

constexpr int kFoldThreads = 128;
constexpr int kPrepassThreads = 128;
constexpr int kPrepassWarps = kPrepassThreads / 32;
constexpr int kXRow = 12;   // 32-bit words per staged input row: 8 half pairs + 4 pad (conflict-free fragment reads)

__global__ void __launch_bounds__(kFoldThreads) k_neural_fold(int64_t n, const __half *__restrict__ features,
                                                              const __half *__restrict__ weights,
                                                              __half *__restrict__ preact) {
  __shared__ float s_w[GS_MLP_HIDDEN][17];   // column 0 and the 16 feature columns of the first layer
  for (int k = threadIdx.x; k < GS_MLP_HIDDEN * 17; k += kFoldThreads) {
    const int o = k / 17, c = k % 17;
    s_w[o][c] = __half2float(weights[kMlpW1 + o * GS_MLP_IN + (c == 0 ? 0 : 15 + c)]);
  }
  __syncthreads();
  const int64_t i = (int64_t)blockIdx.x * kFoldThreads + threadIdx.x;
  if (i >= n) return;
  const uint4 raw = __ldg(reinterpret_cast<const uint4 *>(features) + i);
  const __half2 *h = reinterpret_cast<const __half2 *>(&raw);
  float enc[16];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float2 f = __half22float2(h[j]);
    sincosf(f.x, &enc[4 * j], &enc[4 * j + 1]);
    sincosf(f.y, &enc[4 * j + 2], &enc[4 * j + 3]);
  }
  uint32_t out[8];
#pragma unroll
  for (int o = 0; o < GS_MLP_HIDDEN; o += 2) {
    float a0 = s_w[o][0] * 0.28209479177387814f, a1 = s_w[o + 1][0] * 0.28209479177387814f;
#pragma unroll
    for (int c = 0; c < 16; ++c) {
      a0 = fmaf(s_w[o][1 + c], enc[c], a0);
      a1 = fmaf(s_w[o + 1][1 + c], enc[c], a1);
    }
    const __half2 p = __floats2half2_rn(a0, a1);
    out[o / 2] = *reinterpret_cast<const uint32_t *>(&p);
  }
  uint4 *dst = reinterpret_cast<uint4 *>(preact + 16 * i);
  dst[0] = make_uint4(out[0], out[1], out[2], out[3]);
  dst[1] = make_uint4(out[4], out[5], out[6], out[7]);
}

__device__ __forceinline__ uint32_t pack_half2(float a, float b) {
  const __half2 p = __floats2half2_rn(a, b);
  return *reinterpret_cast<const uint32_t *>(&p);
}
__device__ __forceinline__ uint32_t pack_weights(const __half *w, int idx) {   // w[idx], w[idx + 1]; idx is even
  return __ldg(reinterpret_cast<const uint32_t *>(w + idx));
}

// One warp per 32 Gaussians.  Lane L prepares row L (direction, SH basis, base colour, alpha byte);
// the rows reach the tensor-core fragment layout through a small shared-memory tile; the weights
// live in ten registers per lane for the whole kernel.
__global__ void __launch_bounds__(kPrepassThreads) k_neural_prepass(int64_t n, int deg, int act, const float *__restrict__ means,
                                                                    const float *__restrict__ logits,
                                                                    const float *__restrict__ base_color,
                                                                    const __half *__restrict__ preact,
                                                                    const __half *__restrict__ weights, float ex, float ey,
                                                                    float ez, uchar4 *__restrict__ rgba,
                                                                    float *__restrict__ color) {
  __shared__ uint32_t s_x[kPrepassWarps][32][kXRow];
  __shared__ float s_y[kPrepassWarps][32][3];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, g = lane >> 2, t = lane & 3;
  // B fragments: B[k][nn] = W[nn][k]; b0 holds k = 2t, 2t+1 and b1 k = 2t+8, 2t+9 of column nn = 8 nt + g.
  // Layer 1 keeps only the direction columns 1..15 (column 0 is the folded constant: its weight is dropped).
  uint32_t w1b0[2], w1b1[2], w2b0[2], w2b1[2], w3b0, w3b1;
#pragma unroll
  for (int nt = 0; nt < 2; ++nt) {
    const int nn = nt * 8 + g;
    w1b0[nt] = pack_weights(weights, kMlpW1 + nn * GS_MLP_IN + 2 * t);
    if (t == 0) w1b0[nt] &= 0xffff0000u;
    w1b1[nt] = pack_weights(weights, kMlpW1 + nn * GS_MLP_IN + 2 * t + 8);
    w2b0[nt] = pack_weights(weights, kMlpW2 + nn * GS_MLP_HIDDEN + 2 * t);
    w2b1[nt] = pack_weights(weights, kMlpW2 + nn * GS_MLP_HIDDEN + 2 * t + 8);
  }
  w3b0 = g < 3 ? pack_weights(weights, kMlpW3 + g * GS_MLP_HIDDEN + 2 * t) : 0u;
  w3b1 = g < 3 ? pack_weights(weights, kMlpW3 + g * GS_MLP_HIDDEN + 2 * t + 8) : 0u;
  const int na = (deg + 1) * (deg + 1);

  const int64_t row0 = ((int64_t)blockIdx.x * kPrepassWarps + warp) * 32;
  if (row0 >= n) return;
  const int64_t i = row0 + lane;
  // ---- this lane's Gaussian: direction, direction inputs, base colour, alpha
  float4 c = make_float4(0.f, 0.f, 0.f, 0.f);   // base colour and the alpha texel value
  {
    float Y[16];
#pragma unroll
    for (int k = 0; k < 16; ++k) Y[k] = 0.f;
    if (i < n) {
      const float dx = __ldg(means + 3 * i) - ex, dy = __ldg(means + 3 * i + 1) - ey, dz = __ldg(means + 3 * i + 2) - ez;
      const float inv = rsqrtf(fmaf(dx, dx, fmaf(dy, dy, dz * dz)));
      sh_basis(dx * inv, dy * inv, dz * inv, Y);
      const float o = 1.f / (1.f + __expf(-__ldg(logits + i)));
      c = make_float4(__ldg(base_color + 3 * i), __ldg(base_color + 3 * i + 1), __ldg(base_color + 3 * i + 2),
                      floorf(fmaf(fminf(fmaxf(o, 0.f), 1.f), 255.f, 0.5f)));
    }
    Y[0] = 0.f;   // folded into the pre-activations
#pragma unroll
    for (int k = 0; k < 8; ++k)
      s_x[warp][lane][k] = pack_half2(2 * k < na ? Y[2 * k] : 0.f, 2 * k + 1 < na ? Y[2 * k + 1] : 0.f);
  }
  __syncwarp();
  float y[2][4];
#pragma unroll
  for (int mt = 0; mt < 2; ++mt) {
    const int r0 = mt * 16 + g, r1 = r0 + 8;
    uint32_t a[4] = {s_x[warp][r0][t], s_x[warp][r1][t], s_x[warp][r0][t + 4], s_x[warp][r1][t + 4]};
    // ---- layer 1, accumulators start at the folded pre-activations
    float h[2][4];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      const int64_t ra = row0 + r0 < n ? row0 + r0 : n - 1, rb = row0 + r1 < n ? row0 + r1 : n - 1;
      const uint32_t p0 = __ldg(reinterpret_cast<const uint32_t *>(preact + 16 * ra + nt * 8 + 2 * t));
      const uint32_t p1 = __ldg(reinterpret_cast<const uint32_t *>(preact + 16 * rb + nt * 8 + 2 * t));
      const float2 f0 = __half22float2(*reinterpret_cast<const __half2 *>(&p0));
      const float2 f1 = __half22float2(*reinterpret_cast<const __half2 *>(&p1));
      h[nt][0] = f0.x; h[nt][1] = f0.y; h[nt][2] = f1.x; h[nt][3] = f1.y;
      if (deg > 0) mlp::mma16816(h[nt], a, w1b0[nt], w1b1[nt]);
    }
    // ---- layer 2: the ReLU'd outputs of two column tiles are one A fragment
    a[0] = pack_half2(fmaxf(h[0][0], 0.f), fmaxf(h[0][1], 0.f)); a[1] = pack_half2(fmaxf(h[0][2], 0.f), fmaxf(h[0][3], 0.f));
    a[2] = pack_half2(fmaxf(h[1][0], 0.f), fmaxf(h[1][1], 0.f)); a[3] = pack_half2(fmaxf(h[1][2], 0.f), fmaxf(h[1][3], 0.f));
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      h[nt][0] = h[nt][1] = h[nt][2] = h[nt][3] = 0.f;
      mlp::mma16816(h[nt], a, w2b0[nt], w2b1[nt]);
    }
    // ---- layer 3 (three outputs, padded to eight columns)
    a[0] = pack_half2(fmaxf(h[0][0], 0.f), fmaxf(h[0][1], 0.f)); a[1] = pack_half2(fmaxf(h[0][2], 0.f), fmaxf(h[0][3], 0.f));
    a[2] = pack_half2(fmaxf(h[1][0], 0.f), fmaxf(h[1][1], 0.f)); a[3] = pack_half2(fmaxf(h[1][2], 0.f), fmaxf(h[1][3], 0.f));
    y[mt][0] = y[mt][1] = y[mt][2] = y[mt][3] = 0.f;
    mlp::mma16816(y[mt], a, w3b0, w3b1);
  }
  // ---- the three outputs go back from the fragment layout (lanes t = 0 hold outputs 0, 1 of rows g and
  // g + 8, lanes t = 1 output 2) to one row per lane, so that every lane finishes its own Gaussian
#pragma unroll
  for (int mt = 0; mt < 2; ++mt) {
    if (t == 0) {
      s_y[warp][mt * 16 + g][0] = y[mt][0]; s_y[warp][mt * 16 + g][1] = y[mt][1];
      s_y[warp][mt * 16 + g + 8][0] = y[mt][2]; s_y[warp][mt * 16 + g + 8][1] = y[mt][3];
    } else if (t == 1) {
      s_y[warp][mt * 16 + g][2] = y[mt][0];
      s_y[warp][mt * 16 + g + 8][2] = y[mt][2];
    }
  }
  __syncwarp();
  if (i < n) {
    float col[3];
    unsigned q[3];
#pragma unroll
    for (int ch = 0; ch < 3; ++ch) {
      // tanh(a) = 1 - 2 / (exp(2a) + 1); the fast exponential and division are far inside the texel's step
      const float res = deg > 0 ? 1.f - __fdividef(2.f, __expf(2.f * s_y[warp][lane][ch]) + 1.f) : 0.f;
      col[ch] = color_act_z(act, (ch == 0 ? c.x : ch == 1 ? c.y : c.z) + 0.5f + res);
      q[ch] = (unsigned)floorf(fmaf(fminf(col[ch], 1.f), 255.f, 0.5f));
    }
    rgba[i] = make_uchar4((unsigned char)q[0], (unsigned char)q[1], (unsigned char)q[2], (unsigned char)c.w);
    if (color) { color[3 * i] = col[0]; color[3 * i + 1] = col[1]; color[3 * i + 2] = col[2]; }
  }
}

}  // namespace

int launch_neural_fold(int64_t n, const __half *features, const __half *weights, __half *preact, cudaStream_t st) {
  if (n <= 0) return 0;
  k_neural_fold<<<(unsigned)((n + kFoldThreads - 1) / kFoldThreads), kFoldThreads, 0, st>>>(n, features, weights, preact);
  return 1;
}

int launch_neural_prepass(int64_t n, int deg, int act, const float *means, const float *logits, const float *base_color,
                          const __half *preact, const __half *weights, const float eye[3], uint8_t *rgba, float *color,
                          cudaStream_t st) {
  if (n <= 0) return 0;
  k_neural_prepass<<<(unsigned)((n + kPrepassThreads - 1) / kPrepassThreads), kPrepassThreads, 0, st>>>(
      n, deg, act, means, logits, base_color, preact, weights, eye[0], eye[1], eye[2], reinterpret_cast<uchar4 *>(rgba), color);
  return 1;
}

}  // namespace gs
