// The shared decoder (32 -> 16 ReLU -> 16 ReLU -> 3, Eq. 5-7) on tensor cores, one warp per 32
// Gaussians, forward and backward.
//
// mma.sync m16n8k16 (fp16 x fp16 -> fp32).  Weights are fp16 by definition, so they enter exactly.
// Activations and gradients are fp32; each is split into a high and a low fp16 half
// (x = hi + lo to about 2^-22 relative) and multiplied in two (or, where both operands are split,
// three) MMAs with fp32 accumulation, which keeps the result at fp32-FMA accuracy.
//
// Layout notes (g = lane / 4, t = lane % 4):
//   A (16x16): a0 = (row g, cols 2t,2t+1)  a1 = (row g+8, same)  a2 = (row g, cols 2t+8,2t+9)  a3 = (row g+8, ..)
//   B (16x8):  b0 = (k 2t,2t+1; col g)     b1 = (k 2t+8,2t+9; col g)
//   C (16x8):  c0 = (row g, col 2t) c1 = (row g, col 2t+1) c2 = (row g+8, col 2t) c3 = (row g+8, col 2t+1)
// Two neighbouring C tiles are, packed to half pairs, exactly the A operand of the next layer, so
// the layers chain in registers.  For the weight gradient (a contraction over the 32 Gaussians)
// operands have to be transposed; movmatrix does that on packed 8x8 tiles without shared memory.
#pragma once

#include <cuda_fp16.h>
#include <stdint.h>

#include "gs.h"

namespace gs {
namespace mlp {

constexpr int kXStride = 20;   // 32-bit words per staged input row: 16 half pairs + 4 pad (conflict-free)
constexpr int kGxStride = 20;  // floats per row of the staged input gradient (16 + pad)

// Decoder weights in shared memory: fp16 as given, plus the transposes the backward multiplies by.
struct __align__(16) Weights {
  __half w[GS_MLP_WEIGHTS];        // W1[16][32] | W2[16][16] | W3[3][16]
  __half w1t[32 * 16];             // W1^T: [in][h1]
  __half w2t[16 * 16];             // W2^T: [h1][h2]
  __half w3t[16 * 4];              // W3^T: [h2][out], out padded to 4 with zero
};

// Per-warp staging.
struct __align__(16) WarpStage {
  uint32_t xhi[32 * kXStride];     // inputs, high halves, row = Gaussian, word = column pair
  uint32_t xlo[32 * kXStride];
  float y[32 * 4];                 // layer-3 output to the owner lanes; later dL/dy from them
  float gx[32 * kGxStride];        // dL/dx of the 16 direction inputs, for the owner lanes
  float gf[32 * 8];                // dL/df
};

__device__ __forceinline__ void load_weights(const __half *gw, Weights &W, int tid, int nthreads) {
  for (int k = tid; k < GS_MLP_WEIGHTS; k += nthreads) W.w[k] = gw[k];
  for (int k = tid; k < 32 * 16; k += nthreads) W.w1t[k] = gw[(k & 15) * 32 + (k >> 4)];
  for (int k = tid; k < 16 * 16; k += nthreads) W.w2t[k] = gw[512 + (k & 15) * 16 + (k >> 4)];
  for (int k = tid; k < 16 * 4; k += nthreads) W.w3t[k] = (k & 3) < 3 ? gw[768 + (k & 3) * 16 + (k >> 2)] : __float2half(0.f);
}

__device__ __forceinline__ void mma16816(float c[4], const uint32_t a[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t movm_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}

// Transpose of a low half: nothing to do when operands are not split.
template <bool kSplit>
__device__ __forceinline__ uint32_t movm_lo(uint32_t a) { return kSplit ? movm_trans(a) : 0u; }

// (a, b) -> packed fp16 pairs hi and lo with a = hi.x + lo.x, b = hi.y + lo.y up to ~2^-22.
// kSplit = false is the paper's own precision (Sec. 4: the decoder in half precision): the operand is the
// rounded value alone, lo stays zero and every product that would take it is left out.
template <bool kSplit = true>
__device__ __forceinline__ void split2(float a, float b, uint32_t &hi, uint32_t &lo) {
  const __half2 h = __floats2half2_rn(a, b);
  hi = *reinterpret_cast<const uint32_t *>(&h);
  lo = 0u;
  if (kSplit) {
    const float2 f = __half22float2(h);
    const __half2 l = __floats2half2_rn(a - f.x, b - f.y);
    lo = *reinterpret_cast<const uint32_t *>(&l);
  }
}

__device__ __forceinline__ float2 unsplit(uint32_t hi, uint32_t lo) {
  const float2 a = __half22float2(*reinterpret_cast<const __half2 *>(&hi));
  const float2 b = __half22float2(*reinterpret_cast<const __half2 *>(&lo));
  return make_float2(a.x + b.x, a.y + b.y);
}

// The owner lane (lane = Gaussian row) parks its 32 inputs.  `Stage` is WarpStage or any struct
// that starts with the same xhi / xlo / y members.
template <bool kSplit, class Stage>
__device__ __forceinline__ void stage_inputs(const float x[32], Stage &S, int lane) {
  uint32_t hi[16], lo[16];
#pragma unroll
  for (int p = 0; p < 16; ++p) split2<kSplit>(x[2 * p], x[2 * p + 1], hi[p], lo[p]);
  uint4 *dh = reinterpret_cast<uint4 *>(S.xhi + lane * kXStride), *dl = reinterpret_cast<uint4 *>(S.xlo + lane * kXStride);
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    dh[q] = make_uint4(hi[4 * q], hi[4 * q + 1], hi[4 * q + 2], hi[4 * q + 3]);
    if (kSplit) dl[q] = make_uint4(lo[4 * q], lo[4 * q + 1], lo[4 * q + 2], lo[4 * q + 3]);
  }
}

// A operand (hi and lo) out of two neighbouring C tiles of one 16-row block.
template <bool kSplit>
__device__ __forceinline__ void a_from_c(const float c_lo[4], const float c_hi[4], uint32_t ahi[4], uint32_t alo[4]) {
  split2<kSplit>(c_lo[0], c_lo[1], ahi[0], alo[0]);
  split2<kSplit>(c_lo[2], c_lo[3], ahi[1], alo[1]);
  split2<kSplit>(c_hi[0], c_hi[1], ahi[2], alo[2]);
  split2<kSplit>(c_hi[2], c_hi[3], ahi[3], alo[3]);
}

struct Activations {
  float h1[2][2][4];   // [16-row block][8-column tile][C fragment], after ReLU
  float h2[2][2][4];
};

// Forward of the three layers for the warp's 32 staged rows.  Leaves y (3 values per row) in
// S.y for the owner lanes; returns the hidden activations for the backward.
template <bool kSplit, class Stage>
__device__ __forceinline__ void forward_warp(const Weights &W, Stage &S, int lane, Activations &act) {
  const int g = lane >> 2, t = lane & 3;
  const uint32_t *w32 = reinterpret_cast<const uint32_t *>(W.w);
  __syncwarp();
  // ---- layer 1: [32 x 32] x W1^T
#pragma unroll
  for (int mt = 0; mt < 2; ++mt)
#pragma unroll
    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
      for (int k = 0; k < 4; ++k) act.h1[mt][nt][k] = 0.f;
#pragma unroll
  for (int ks = 0; ks < 2; ++ks) {
    uint32_t b0[2], b1[2];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      const int word = ((8 * nt + g) * 32 + 16 * ks + 2 * t) >> 1;
      b0[nt] = w32[word]; b1[nt] = w32[word + 4];
    }
#pragma unroll
    for (int mt = 0; mt < 2; ++mt) {
      const int r0 = (16 * mt + g) * kXStride + 8 * ks + t, r1 = r0 + 8 * kXStride;
      const uint32_t ahi[4] = {S.xhi[r0], S.xhi[r1], S.xhi[r0 + 4], S.xhi[r1 + 4]};
      uint32_t alo[4] = {0u, 0u, 0u, 0u};
      if (kSplit) { alo[0] = S.xlo[r0]; alo[1] = S.xlo[r1]; alo[2] = S.xlo[r0 + 4]; alo[3] = S.xlo[r1 + 4]; }
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        mma16816(act.h1[mt][nt], ahi, b0[nt], b1[nt]);
        if (kSplit) mma16816(act.h1[mt][nt], alo, b0[nt], b1[nt]);
      }
    }
  }
#pragma unroll
  for (int mt = 0; mt < 2; ++mt)
#pragma unroll
    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
      for (int k = 0; k < 4; ++k) act.h1[mt][nt][k] = fmaxf(act.h1[mt][nt][k], 0.f);
  // ---- layer 2: [32 x 16] x W2^T
  {
    uint32_t b0[2], b1[2];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      const int word = 256 + (((8 * nt + g) * 16 + 2 * t) >> 1);
      b0[nt] = w32[word]; b1[nt] = w32[word + 4];
    }
#pragma unroll
    for (int mt = 0; mt < 2; ++mt) {
      uint32_t ahi[4], alo[4];
      a_from_c<kSplit>(act.h1[mt][0], act.h1[mt][1], ahi, alo);
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
        for (int k = 0; k < 4; ++k) act.h2[mt][nt][k] = 0.f;
        mma16816(act.h2[mt][nt], ahi, b0[nt], b1[nt]);
        if (kSplit) mma16816(act.h2[mt][nt], alo, b0[nt], b1[nt]);
      }
    }
  }
#pragma unroll
  for (int mt = 0; mt < 2; ++mt)
#pragma unroll
    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
      for (int k = 0; k < 4; ++k) act.h2[mt][nt][k] = fmaxf(act.h2[mt][nt][k], 0.f);
  // ---- layer 3: [32 x 16] x W3^T (3 outputs, padded to 8)
  {
    const int word = 384 + ((g * 16 + 2 * t) >> 1);
    const uint32_t b0 = g < 3 ? w32[word] : 0u, b1 = g < 3 ? w32[word + 4] : 0u;
#pragma unroll
    for (int mt = 0; mt < 2; ++mt) {
      uint32_t ahi[4], alo[4];
      a_from_c<kSplit>(act.h2[mt][0], act.h2[mt][1], ahi, alo);
      float c[4] = {0.f, 0.f, 0.f, 0.f};
      mma16816(c, ahi, b0, b1);
      if (kSplit) mma16816(c, alo, b0, b1);
      const int r0 = (16 * mt + g) * 4, r1 = r0 + 32;
      if (t == 0) { S.y[r0] = c[0]; S.y[r0 + 1] = c[1]; S.y[r1] = c[2]; S.y[r1 + 1] = c[3]; }
      if (t == 1) { S.y[r0 + 2] = c[0]; S.y[r1 + 2] = c[2]; }
    }
  }
  __syncwarp();
}

// Weight-gradient accumulators of one warp, as C fragments: dW1 [16 x 32] in four column tiles,
// dW2 [16 x 16] in two, dW3 [3 (of 16) x 16] in two.
struct WeightGrad {
  float w1[4][4], w2[2][4], w3[2][4];
  __device__ __forceinline__ void clear() {
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int k = 0; k < 4; ++k) w1[a][k] = 0.f;
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
      for (int k = 0; k < 4; ++k) { w2[a][k] = 0.f; w3[a][k] = 0.f; }
  }
};

// c += A^T-style product with both operands split: (Ahi + Alo)(Bhi + Blo) without the lo*lo term.
template <bool kSplit>
__device__ __forceinline__ void mma3(float c[4], const uint32_t ahi[4], const uint32_t alo[4], uint32_t b0h, uint32_t b1h,
                                     uint32_t b0l, uint32_t b1l) {
  mma16816(c, ahi, b0h, b1h);
  if (kSplit) {
    mma16816(c, ahi, b0l, b1l);
    mma16816(c, alo, b0h, b1h);
  }
}

// Backward of the three layers.  On entry the owner lanes have written dL/dy (3 values per row,
// 4th = 0) into S.y.  On exit S.gx holds dL/dx of the 16 direction inputs and S.gf holds dL/df per
// row, and the warp's weight-gradient fragments have been advanced.
template <bool kSplit>
__device__ __forceinline__ void backward_warp(const Weights &W, WarpStage &S, int lane, const Activations &act,
                                              WeightGrad &dW) {
  const int g = lane >> 2, t = lane & 3;
  __syncwarp();
  // ---- dL/dh2 = gY W3, masked by h2 > 0
  float d2[2][2][4], d1[2][2][4];
  {
    const uint32_t *w3t = reinterpret_cast<const uint32_t *>(W.w3t);
    uint32_t b0[2];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) b0[nt] = t < 2 ? w3t[(8 * nt + g) * 2 + t] : 0u;
#pragma unroll
    for (int mt = 0; mt < 2; ++mt) {
      uint32_t ahi[4] = {0u, 0u, 0u, 0u}, alo[4] = {0u, 0u, 0u, 0u};
      if (t < 2) {
        const float2 u0 = *reinterpret_cast<const float2 *>(S.y + (16 * mt + g) * 4 + 2 * t);
        const float2 u1 = *reinterpret_cast<const float2 *>(S.y + (16 * mt + g + 8) * 4 + 2 * t);
        split2<kSplit>(u0.x, u0.y, ahi[0], alo[0]);
        split2<kSplit>(u1.x, u1.y, ahi[1], alo[1]);
      }
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
        for (int k = 0; k < 4; ++k) d2[mt][nt][k] = 0.f;
        mma16816(d2[mt][nt], ahi, b0[nt], 0u);
        if (kSplit) mma16816(d2[mt][nt], alo, b0[nt], 0u);
#pragma unroll
        for (int k = 0; k < 4; ++k) d2[mt][nt][k] = act.h2[mt][nt][k] > 0.f ? d2[mt][nt][k] : 0.f;
      }
    }
  }
  // ---- dL/dh1 = d2 W2, masked by h1 > 0
  {
    const uint32_t *w2t = reinterpret_cast<const uint32_t *>(W.w2t);
    uint32_t b0[2], b1[2];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      const int word = ((8 * nt + g) * 16 + 2 * t) >> 1;
      b0[nt] = w2t[word]; b1[nt] = w2t[word + 4];
    }
#pragma unroll
    for (int mt = 0; mt < 2; ++mt) {
      uint32_t ahi[4], alo[4];
      a_from_c<kSplit>(d2[mt][0], d2[mt][1], ahi, alo);
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
        for (int k = 0; k < 4; ++k) d1[mt][nt][k] = 0.f;
        mma16816(d1[mt][nt], ahi, b0[nt], b1[nt]);
        if (kSplit) mma16816(d1[mt][nt], alo, b0[nt], b1[nt]);
#pragma unroll
        for (int k = 0; k < 4; ++k) d1[mt][nt][k] = act.h1[mt][nt][k] > 0.f ? d1[mt][nt][k] : 0.f;
      }
    }
  }
  // ---- dL/dx = d1 W1: columns 0..15 (directions) to S.gx, columns 16..31 (sin, cos pairs) to dL/df
  {
    const uint32_t *w1t = reinterpret_cast<const uint32_t *>(W.w1t);
#pragma unroll
    for (int mt = 0; mt < 2; ++mt) {
      uint32_t ahi[4], alo[4];
      a_from_c<kSplit>(d1[mt][0], d1[mt][1], ahi, alo);
      const int r0 = 16 * mt + g, r1 = r0 + 8;
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        const int word = ((8 * nt + g) * 16 + 2 * t) >> 1;
        const uint32_t b0 = w1t[word], b1 = w1t[word + 4];
        float c[4] = {0.f, 0.f, 0.f, 0.f};
        mma16816(c, ahi, b0, b1);
        if (kSplit) mma16816(c, alo, b0, b1);
        if (nt < 2) {
          *reinterpret_cast<float2 *>(S.gx + r0 * kGxStride + 8 * nt + 2 * t) = make_float2(c[0], c[1]);
          *reinterpret_cast<float2 *>(S.gx + r1 * kGxStride + 8 * nt + 2 * t) = make_float2(c[2], c[3]);
        } else {
          // columns 16 + 2j, 17 + 2j are (sin f_j, cos f_j) with j = 4 (nt - 2) + t
          const int j = 4 * (nt - 2) + t;
          const float2 sc0 = unsplit(S.xhi[r0 * kXStride + 8 + j], kSplit ? S.xlo[r0 * kXStride + 8 + j] : 0u);
          const float2 sc1 = unsplit(S.xhi[r1 * kXStride + 8 + j], kSplit ? S.xlo[r1 * kXStride + 8 + j] : 0u);
          S.gf[r0 * 8 + j] = c[0] * sc0.y - c[1] * sc0.x;
          S.gf[r1 * 8 + j] = c[2] * sc1.y - c[3] * sc1.x;
        }
      }
    }
  }
  // ---- weight gradients: contractions over the 32 Gaussians (two k-steps of 16 rows)
#pragma unroll
  for (int ks = 0; ks < 2; ++ks) {
    // dW3 += gY^T H2
    {
      uint32_t ahi[4] = {0u, 0u, 0u, 0u}, alo[4] = {0u, 0u, 0u, 0u};
      if (g < 3) {
        const int ra = (16 * ks + 2 * t) * 4 + g;
        split2<kSplit>(S.y[ra], S.y[ra + 4], ahi[0], alo[0]);
        split2<kSplit>(S.y[ra + 32], S.y[ra + 36], ahi[2], alo[2]);
      }
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        uint32_t th, tl, bh, bl;
        split2<kSplit>(act.h2[ks][nt][0], act.h2[ks][nt][1], th, tl);
        split2<kSplit>(act.h2[ks][nt][2], act.h2[ks][nt][3], bh, bl);
        mma3<kSplit>(dW.w3[nt], ahi, alo, movm_trans(th), movm_trans(bh), movm_lo<kSplit>(tl), movm_lo<kSplit>(bl));
      }
    }
    // dW2 += d2^T H1
    {
      uint32_t ahi[4], alo[4];
      {
        uint32_t h, l;
        split2<kSplit>(d2[ks][0][0], d2[ks][0][1], h, l); ahi[0] = movm_trans(h); alo[0] = movm_lo<kSplit>(l);
        split2<kSplit>(d2[ks][1][0], d2[ks][1][1], h, l); ahi[1] = movm_trans(h); alo[1] = movm_lo<kSplit>(l);
        split2<kSplit>(d2[ks][0][2], d2[ks][0][3], h, l); ahi[2] = movm_trans(h); alo[2] = movm_lo<kSplit>(l);
        split2<kSplit>(d2[ks][1][2], d2[ks][1][3], h, l); ahi[3] = movm_trans(h); alo[3] = movm_lo<kSplit>(l);
      }
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        uint32_t th, tl, bh, bl;
        split2<kSplit>(act.h1[ks][nt][0], act.h1[ks][nt][1], th, tl);
        split2<kSplit>(act.h1[ks][nt][2], act.h1[ks][nt][3], bh, bl);
        mma3<kSplit>(dW.w2[nt], ahi, alo, movm_trans(th), movm_trans(bh), movm_lo<kSplit>(tl), movm_lo<kSplit>(bl));
      }
    }
    // dW1 += d1^T X
    {
      uint32_t ahi[4], alo[4];
      {
        uint32_t h, l;
        split2<kSplit>(d1[ks][0][0], d1[ks][0][1], h, l); ahi[0] = movm_trans(h); alo[0] = movm_lo<kSplit>(l);
        split2<kSplit>(d1[ks][1][0], d1[ks][1][1], h, l); ahi[1] = movm_trans(h); alo[1] = movm_lo<kSplit>(l);
        split2<kSplit>(d1[ks][0][2], d1[ks][0][3], h, l); ahi[2] = movm_trans(h); alo[2] = movm_lo<kSplit>(l);
        split2<kSplit>(d1[ks][1][2], d1[ks][1][3], h, l); ahi[3] = movm_trans(h); alo[3] = movm_lo<kSplit>(l);
      }
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        // the 8 x 8 tile X[rows 16ks + (0..7 | 8..15)][cols 8nt .. 8nt+7] as packed pairs, then transposed
        const int r0 = (16 * ks + g) * kXStride + 4 * nt + t, r1 = r0 + 8 * kXStride;
        mma3<kSplit>(dW.w1[nt], ahi, alo, movm_trans(S.xhi[r0]), movm_trans(S.xhi[r1]), movm_lo<kSplit>(kSplit ? S.xlo[r0] : 0u),
                     movm_lo<kSplit>(kSplit ? S.xlo[r1] : 0u));
      }
    }
  }
  __syncwarp();
}

// Write one warp's weight-gradient fragments into a [816] fp32 array (W1 | W2 | W3 layout).
__device__ __forceinline__ void store_weight_grad(const WeightGrad &dW, float *part, int lane) {
  const int g = lane >> 2, t = lane & 3;
#pragma unroll
  for (int nt = 0; nt < 4; ++nt) {
    float *p = part + g * 32 + 8 * nt + 2 * t;
    p[0] = dW.w1[nt][0]; p[1] = dW.w1[nt][1]; p[8 * 32] = dW.w1[nt][2]; p[8 * 32 + 1] = dW.w1[nt][3];
  }
#pragma unroll
  for (int nt = 0; nt < 2; ++nt) {
    float *p = part + 512 + g * 16 + 8 * nt + 2 * t;
    p[0] = dW.w2[nt][0]; p[1] = dW.w2[nt][1]; p[8 * 16] = dW.w2[nt][2]; p[8 * 16 + 1] = dW.w2[nt][3];
    if (g < 3) {
      float *q = part + 768 + g * 16 + 8 * nt + 2 * t;
      q[0] = dW.w3[nt][0]; q[1] = dW.w3[nt][1];
    }
  }
}

}  // namespace mlp
}  // namespace gs
