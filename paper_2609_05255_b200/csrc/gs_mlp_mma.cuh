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
// the layers chain in registers; and the packed pairs are what is kept of a layer (not the fp32
// values): the backward takes its ReLU masks from them and, transposed, the operands of the weight
// gradient, without splitting anything a second time.  The weight gradient contracts over the 32
// Gaussians, so one operand of each product has to be transposed: movmatrix does that for values
// that live in registers, ldmatrix.trans for the staged inputs.
#pragma once

#include <cuda_fp16.h>
#include <stdint.h>

#include "gs.h"

namespace gs {
namespace mlp {

constexpr int kXStride = 20;   // 32-bit words per staged input row: 16 half pairs + 4 pad (80-byte rows: 16-byte aligned
                               // for ldmatrix, and eight consecutive rows fall into different banks)
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

// The forward's B operands, as each lane holds them: 14 registers, read once by a kernel that decodes many rows.
struct FwdFrags {
  uint32_t w1[2][2][2];   // [k-step][column tile][b0, b1]
  uint32_t w2[2][2];      // [column tile][b0, b1]
  uint32_t w3[2];
};
// `gw`: the 816 weights as given (global or shared memory, 4-byte aligned).
__device__ __forceinline__ FwdFrags load_fwd_frags(const __half *gw, int lane) {
  const int g = lane >> 2, t = lane & 3;
  const uint32_t *w32 = reinterpret_cast<const uint32_t *>(gw);
  FwdFrags F;
#pragma unroll
  for (int ks = 0; ks < 2; ++ks)
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      const int word = ((8 * nt + g) * 32 + 16 * ks + 2 * t) >> 1;
      F.w1[ks][nt][0] = w32[word]; F.w1[ks][nt][1] = w32[word + 4];
    }
#pragma unroll
  for (int nt = 0; nt < 2; ++nt) {
    const int word = 256 + (((8 * nt + g) * 16 + 2 * t) >> 1);
    F.w2[nt][0] = w32[word]; F.w2[nt][1] = w32[word + 4];
  }
  const int word = 384 + ((g * 16 + 2 * t) >> 1);
  F.w3[0] = g < 3 ? w32[word] : 0u;
  F.w3[1] = g < 3 ? w32[word + 4] : 0u;
  return F;
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

// Four 8x8 tiles of 16-bit values out of shared memory in one instruction; lane i passes the address of row i % 8 of
// tile i / 8 (16 bytes, 16-byte aligned), and register k of lane (g, t) receives elements (g; 2t, 2t+1) of tile k -
// or, transposed, elements (2t, 2t+1; g).
__device__ __forceinline__ void ldsm_x4(uint32_t r[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t r[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

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

// A operand (hi and lo) out of two neighbouring C tiles of one 16-row block; with kRelu the values pass max(., 0) first.
template <bool kSplit, bool kRelu>
__device__ __forceinline__ void a_from_c(const float c_lo[4], const float c_hi[4], uint32_t ahi[4], uint32_t alo[4]) {
  float u[4], v[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) { u[k] = kRelu ? fmaxf(c_lo[k], 0.f) : c_lo[k]; v[k] = kRelu ? fmaxf(c_hi[k], 0.f) : c_hi[k]; }
  split2<kSplit>(u[0], u[1], ahi[0], alo[0]);
  split2<kSplit>(u[2], u[3], ahi[1], alo[1]);
  split2<kSplit>(v[0], v[1], ahi[2], alo[2]);
  split2<kSplit>(v[2], v[3], ahi[3], alo[3]);
}

// The hidden activations (after ReLU) of the warp's 32 rows as packed A operands: [16-row block][a0..a3].
struct Activations {
  uint32_t h1hi[2][4], h1lo[2][4], h2hi[2][4], h2lo[2][4];
};

// dL/d(pre-activation) from dL/d(activation): the C tile pair (columns 0..7, 8..15) of one 16-row block keeps its value
// where the activation, read from the high halves of its packed A operand, is positive.
__device__ __forceinline__ void relu_mask(float c_lo[4], float c_hi[4], const uint32_t ahi[4]) {
  c_lo[0] = (ahi[0] & 0xffffu) ? c_lo[0] : 0.f; c_lo[1] = (ahi[0] >> 16) ? c_lo[1] : 0.f;
  c_lo[2] = (ahi[1] & 0xffffu) ? c_lo[2] : 0.f; c_lo[3] = (ahi[1] >> 16) ? c_lo[3] : 0.f;
  c_hi[0] = (ahi[2] & 0xffffu) ? c_hi[0] : 0.f; c_hi[1] = (ahi[2] >> 16) ? c_hi[1] : 0.f;
  c_hi[2] = (ahi[3] & 0xffffu) ? c_hi[2] : 0.f; c_hi[3] = (ahi[3] >> 16) ? c_hi[3] : 0.f;
}

// Forward of the three layers for the warp's 32 staged rows.  Leaves y (3 values per row) in
// S.y for the owner lanes; returns the hidden activations for the backward.
template <bool kSplit, class Stage>
__device__ __forceinline__ void forward_warp(const FwdFrags &F, Stage &S, int lane, Activations &act) {
  const int g = lane >> 2, t = lane & 3;
  __syncwarp();
  // ---- layer 1: [32 x 32] x W1^T; the A operands come out of the staged rows one 16 x 16 block per instruction
  float c1[2][2][4];
#pragma unroll
  for (int mt = 0; mt < 2; ++mt)
#pragma unroll
    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
      for (int k = 0; k < 4; ++k) c1[mt][nt][k] = 0.f;
  {
    const int tile = lane >> 3, r = lane & 7;
    const uint32_t lane_off = (uint32_t)((r + 8 * (tile & 1)) * kXStride * 4 + (tile >> 1) * 16);
    const uint32_t hi_base = smem_u32(S.xhi) + lane_off, lo_base = smem_u32(S.xlo) + lane_off;
#pragma unroll
    for (int ks = 0; ks < 2; ++ks)
#pragma unroll
      for (int mt = 0; mt < 2; ++mt) {
        const uint32_t off = (uint32_t)(mt * 16 * kXStride * 4 + ks * 32);
        uint32_t ahi[4], alo[4];
        ldsm_x4(ahi, hi_base + off);
        if (kSplit) ldsm_x4(alo, lo_base + off);
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
          mma16816(c1[mt][nt], ahi, F.w1[ks][nt][0], F.w1[ks][nt][1]);
          if (kSplit) mma16816(c1[mt][nt], alo, F.w1[ks][nt][0], F.w1[ks][nt][1]);
        }
      }
  }
#pragma unroll
  for (int mt = 0; mt < 2; ++mt) {
    a_from_c<kSplit, true>(c1[mt][0], c1[mt][1], act.h1hi[mt], act.h1lo[mt]);
    // ---- layer 2: [32 x 16] x W2^T
    float c2[2][4];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
      for (int k = 0; k < 4; ++k) c2[nt][k] = 0.f;
      mma16816(c2[nt], act.h1hi[mt], F.w2[nt][0], F.w2[nt][1]);
      if (kSplit) mma16816(c2[nt], act.h1lo[mt], F.w2[nt][0], F.w2[nt][1]);
    }
    a_from_c<kSplit, true>(c2[0], c2[1], act.h2hi[mt], act.h2lo[mt]);
    // ---- layer 3: [32 x 16] x W3^T (3 outputs, padded to 8)
    float c[4] = {0.f, 0.f, 0.f, 0.f};
    mma16816(c, act.h2hi[mt], F.w3[0], F.w3[1]);
    if (kSplit) mma16816(c, act.h2lo[mt], F.w3[0], F.w3[1]);
    const int r0 = (16 * mt + g) * 4, r1 = r0 + 32;
    if (t == 0) { S.y[r0] = c[0]; S.y[r0 + 1] = c[1]; S.y[r1] = c[2]; S.y[r1 + 1] = c[3]; }
    if (t == 1) { S.y[r0 + 2] = c[0]; S.y[r1 + 2] = c[2]; }
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

// A packed A operand of 16 rows x 16 columns, transposed: the A operand of the product that contracts over those rows.
template <bool kSplit>
__device__ __forceinline__ void transpose_a(const uint32_t hi[4], const uint32_t lo[4], uint32_t thi[4], uint32_t tlo[4]) {
  // tiles: [0] rows 0..7 / cols 0..7, [1] rows 8..15 / cols 0..7, [2] rows 0..7 / cols 8..15, [3] rows 8..15 / cols 8..15;
  // transposing the block swaps the off-diagonal tiles
  thi[0] = movm_trans(hi[0]); thi[1] = movm_trans(hi[2]); thi[2] = movm_trans(hi[1]); thi[3] = movm_trans(hi[3]);
  tlo[0] = movm_lo<kSplit>(lo[0]); tlo[1] = movm_lo<kSplit>(lo[2]); tlo[2] = movm_lo<kSplit>(lo[1]); tlo[3] = movm_lo<kSplit>(lo[3]);
}

// Backward of the three layers.  On entry the owner lanes have written dL/dy (3 values per row,
// 4th = 0) into S.y.  On exit S.gx holds dL/dx of the 16 direction inputs and S.gf holds dL/df per
// row, and the warp's weight-gradient fragments have been advanced.
template <bool kSplit>
__device__ __forceinline__ void backward_warp(const Weights &W, WarpStage &S, int lane, const Activations &act,
                                              WeightGrad &dW) {
  const int g = lane >> 2, t = lane & 3;
  __syncwarp();
  const uint32_t *w3t = reinterpret_cast<const uint32_t *>(W.w3t);
  const uint32_t *w2t = reinterpret_cast<const uint32_t *>(W.w2t);
  const uint32_t *w1t = reinterpret_cast<const uint32_t *>(W.w1t);
  const int tile = lane >> 3, r = lane & 7;
  const uint32_t xhi_base = smem_u32(S.xhi), xlo_base = smem_u32(S.xlo);
#pragma unroll
  for (int mt = 0; mt < 2; ++mt) {   // one 16-row block at a time: it is also one k-step of the weight gradients
    // ---- dL/dy of the block as an A operand (rows g, g+8; columns 0..3 of 16), and transposed for dW3
    uint32_t yhi[4] = {0u, 0u, 0u, 0u}, ylo[4] = {0u, 0u, 0u, 0u};
    if (t < 2) {
      const float2 u0 = *reinterpret_cast<const float2 *>(S.y + (16 * mt + g) * 4 + 2 * t);
      const float2 u1 = *reinterpret_cast<const float2 *>(S.y + (16 * mt + g + 8) * 4 + 2 * t);
      split2<kSplit>(u0.x, u0.y, yhi[0], ylo[0]);
      split2<kSplit>(u1.x, u1.y, yhi[1], ylo[1]);
    }
    // ---- dL/dh2 = gY W3, masked by h2 > 0
    float d2[2][4];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      const uint32_t b0 = t < 2 ? w3t[(8 * nt + g) * 2 + t] : 0u;
#pragma unroll
      for (int k = 0; k < 4; ++k) d2[nt][k] = 0.f;
      mma16816(d2[nt], yhi, b0, 0u);
      if (kSplit) mma16816(d2[nt], ylo, b0, 0u);
    }
    relu_mask(d2[0], d2[1], act.h2hi[mt]);
    uint32_t d2hi[4], d2lo[4];
    a_from_c<kSplit, false>(d2[0], d2[1], d2hi, d2lo);
    // ---- dL/dh1 = d2 W2, masked by h1 > 0
    float d1[2][4];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      const int word = ((8 * nt + g) * 16 + 2 * t) >> 1;
#pragma unroll
      for (int k = 0; k < 4; ++k) d1[nt][k] = 0.f;
      mma16816(d1[nt], d2hi, w2t[word], w2t[word + 4]);
      if (kSplit) mma16816(d1[nt], d2lo, w2t[word], w2t[word + 4]);
    }
    relu_mask(d1[0], d1[1], act.h1hi[mt]);
    uint32_t d1hi[4], d1lo[4];
    a_from_c<kSplit, false>(d1[0], d1[1], d1hi, d1lo);
    // ---- dL/dx = d1 W1: columns 0..15 (directions) to S.gx, columns 16..31 (sin, cos pairs) to dL/df
    {
      const int r0 = 16 * mt + g, r1 = r0 + 8;
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        const int word = ((8 * nt + g) * 16 + 2 * t) >> 1;
        const uint32_t b0 = w1t[word], b1 = w1t[word + 4];
        float c[4] = {0.f, 0.f, 0.f, 0.f};
        mma16816(c, d1hi, b0, b1);
        if (kSplit) mma16816(c, d1lo, b0, b1);
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
    // ---- weight gradients: the block's 16 Gaussians are one k-step of each contraction
    // dW3 += gY^T H2   (gY^T: 3 of 16 rows)
    {
      uint32_t ahi[4] = {0u, 0u, 0u, 0u}, alo[4] = {0u, 0u, 0u, 0u};
      if (g < 3) {
        const int ra = (16 * mt + 2 * t) * 4 + g;
        split2<kSplit>(S.y[ra], S.y[ra + 4], ahi[0], alo[0]);
        split2<kSplit>(S.y[ra + 32], S.y[ra + 36], ahi[2], alo[2]);
      }
#pragma unroll
      for (int nt = 0; nt < 2; ++nt)
        mma3<kSplit>(dW.w3[nt], ahi, alo, movm_trans(act.h2hi[mt][2 * nt]), movm_trans(act.h2hi[mt][2 * nt + 1]),
                     movm_lo<kSplit>(act.h2lo[mt][2 * nt]), movm_lo<kSplit>(act.h2lo[mt][2 * nt + 1]));
    }
    // dW2 += d2^T H1
    {
      uint32_t ahi[4], alo[4];
      transpose_a<kSplit>(d2hi, d2lo, ahi, alo);
#pragma unroll
      for (int nt = 0; nt < 2; ++nt)
        mma3<kSplit>(dW.w2[nt], ahi, alo, movm_trans(act.h1hi[mt][2 * nt]), movm_trans(act.h1hi[mt][2 * nt + 1]),
                     movm_lo<kSplit>(act.h1lo[mt][2 * nt]), movm_lo<kSplit>(act.h1lo[mt][2 * nt + 1]));
    }
    // dW1 += d1^T X: the staged rows of the block, transposed on their way out of shared memory (two column tiles
    // per instruction: b0, b1 of tile nt and of tile nt + 1)
    {
      uint32_t ahi[4], alo[4];
      transpose_a<kSplit>(d1hi, d1lo, ahi, alo);
      const uint32_t lane_off = (uint32_t)((16 * mt + r + 8 * (tile & 1)) * kXStride * 4 + (tile >> 1) * 16);
#pragma unroll
      for (int np = 0; np < 2; ++np) {
        uint32_t bh[4], bl[4] = {0u, 0u, 0u, 0u};
        ldsm_x4_trans(bh, xhi_base + lane_off + np * 32);
        if (kSplit) ldsm_x4_trans(bl, xlo_base + lane_off + np * 32);
        mma3<kSplit>(dW.w1[2 * np], ahi, alo, bh[0], bh[1], bl[0], bl[1]);
        mma3<kSplit>(dW.w1[2 * np + 1], ahi, alo, bh[2], bh[3], bl[2], bl[3]);
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
